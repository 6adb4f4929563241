#include <type_traits>
// Dense linear algebra behind Eq. 3-5 / 3-6: the eigen-decomposition of the Gram matrix
// G = O O^T = U Sigma^2 U^T, which yields the singular values and the rows of U Sigma that the
// information contribution score sums.
//
// Two routes, chosen by rank_cap:
//   full      one-sided Jacobi on the N x N matrix (columns of W = G J are orthogonalised; the
//             accumulated rotations J are the eigenvectors, the column norms the eigenvalues).
//   subspace  when the caller bounds the numerical rank by k < N: a k-dimensional dominant
//             subspace is built (sign sketch of O, one multiplication by G, Cholesky-QR
//             orthonormalisation), G is projected onto it (Rayleigh-Ritz) and only the k x k
//             projection goes through Jacobi, inside shared memory.
// All arithmetic is float32 with a fixed summation order.
#include "tc_internal.cuh"

namespace tc {

// 16-byte asynchronous copy global -> shared; `bytes` = 16, or 0 to write zeros instead.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc, int bytes) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(gsrc), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}


// ==========================================================================================
// Batched float32 GEMM on the plain ALUs:  C[m][n] = sum_k opA[m][k] * opB[k][n].
//   opA[m][k] = TRA ? A[k * lda + m] : A[m * lda + k]
//   opB[k][n] = TRB ? B[n * ldb + k] : B[k * ldb + n]
// 64 x 64 tile per block, 16-deep slices, 4 x 4 outputs per thread.  blockIdx.z = batch.
// ==========================================================================================
__device__ inline float ld_f32(const float* p) { return __ldg(p); }
__device__ inline float ld_f32(const __half* p) { return __half2float(__ldg(p)); }
__device__ inline float ld_f32(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// flags for structured products
constexpr int GEMM_SYM = 1;       // C is symmetric (A^T A): tiles below the diagonal are mirrored
constexpr int GEMM_B_UPPER = 2;   // opB[k][n] = 0 for k > n: the K loop stops at the tile's edge

template <typename TA, typename TB, bool TRA, bool TRB, int RM, int CN>
__global__ void __launch_bounds__(256) gemm_kernel(const TA* __restrict__ A,
                                                  const TB* __restrict__ B, float* __restrict__ C,
                                                  int M, int N, int K, int lda, int ldb, int ldc,
                                                  size_t sA, size_t sB, size_t sC, int flags) {
  // (64 RM) x (16 CN) tile per block, 16-deep slices, (4 RM) x CN outputs per thread.  The next
  // slice is fetched into registers while the current one is multiplied out of shared memory.
  // CN = 4 gives 64-column tiles, CN = 3 gives 48-column tiles (for widths like 144 = 3 * 48).
  constexpr int BM = 64 * RM, BN = 16 * CN, BK = 16;
  constexpr int LA = BM * BK / 256, LB = BN * BK / 256;
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  if ((flags & GEMM_SYM) && n0 + BN <= m0) return;  // strictly below the diagonal
  A += (size_t)blockIdx.z * sA;
  B += (size_t)blockIdx.z * sB;
  C += (size_t)blockIdx.z * sC;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int Kend = (flags & GEMM_B_UPPER) ? min(K, n0 + BN) : K;
  float acc[4 * RM][CN];
#pragma unroll
  for (int i = 0; i < 4 * RM; ++i)
#pragma unroll
    for (int j = 0; j < CN; ++j) acc[i][j] = 0.f;
  // Slices are fetched as 16-byte vectors along the contiguous direction of each operand when
  // every address involved is 16-byte aligned (float32 operands, leading dimensions, sizes and
  // batch strides multiples of four); otherwise element by element.
  constexpr bool F32 = (sizeof(TA) == 4) && (sizeof(TB) == 4);
  const bool vec = F32 && ((lda | ldb | M | N | K) & 3) == 0 && ((sA | sB) & 3) == 0 &&
                   ((((uintptr_t)A) | ((uintptr_t)B)) & 15) == 0;
  constexpr int VA = LA / 4, VB = (LB + 3) / 4;  // vectors per thread (B: some threads idle)
  float ra[LA], rb[VB * 4];

  auto fetch = [&](int k0) {
    if (vec) {
#pragma unroll
      for (int i = 0; i < VA; ++i) {
        const int e = tid + i * 256;  // vector index inside the A slice
        int m, k;
        if (TRA) {  // stored [k][m]: vectors run along m
          m = (e % (BM / 4)) * 4;
          k = e / (BM / 4);
        } else {  // stored [m][k]: vectors run along k
          k = (e & 3) * 4;
          m = e >> 2;
        }
        const int gm = m0 + m, gk = k0 + k;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (gm < M && gk < Kend)
          v = __ldg(reinterpret_cast<const float4*>(
              TRA ? (const float*)A + (size_t)gk * lda + gm : (const float*)A + (size_t)gm * lda + gk));
        ra[4 * i] = v.x; ra[4 * i + 1] = v.y; ra[4 * i + 2] = v.z; ra[4 * i + 3] = v.w;
      }
#pragma unroll
      for (int i = 0; i < VB; ++i) {
        const int e = tid + i * 256;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (e < BN * BK / 4) {
          int n, k;
          if (TRB) {  // stored [n][k]: vectors run along k
            k = (e & 3) * 4;
            n = e >> 2;
          } else {  // stored [k][n]: vectors run along n
            n = (e % (BN / 4)) * 4;
            k = e / (BN / 4);
          }
          const int gn = n0 + n, gk = k0 + k;
          if (gn < N && gk < Kend)
            v = __ldg(reinterpret_cast<const float4*>(
                TRB ? (const float*)B + (size_t)gn * ldb + gk : (const float*)B + (size_t)gk * ldb + gn));
        }
        rb[4 * i] = v.x; rb[4 * i + 1] = v.y; rb[4 * i + 2] = v.z; rb[4 * i + 3] = v.w;
      }
      return;
    }
#pragma unroll
    for (int i = 0; i < LA; ++i) {
      const int e = tid + i * 256;
      int m, k;
      if (TRA) {
        m = e % BM;
        k = e / BM;
      } else {
        k = e & 15;
        m = e >> 4;
      }
      const int gm = m0 + m, gk = k0 + k;
      float v = 0.f;
      if (gm < M && gk < Kend) v = TRA ? ld_f32(A + (size_t)gk * lda + gm) : ld_f32(A + (size_t)gm * lda + gk);
      ra[i] = v;
    }
#pragma unroll
    for (int i = 0; i < LB; ++i) {
      const int e = tid + i * 256;
      int n, k;
      if (TRB) {
        k = e & 15;
        n = e >> 4;
      } else {
        n = e % BN;
        k = e / BN;
      }
      const int gn = n0 + n, gk = k0 + k;
      float v = 0.f;
      if (gn < N && gk < Kend) v = TRB ? ld_f32(B + (size_t)gn * ldb + gk) : ld_f32(B + (size_t)gk * ldb + gn);
      rb[i] = v;
    }
  };
  auto stash = [&]() {
    if (vec) {
#pragma unroll
      for (int i = 0; i < VA; ++i) {
        const int e = tid + i * 256;
        if (TRA) {
          const int m = (e % (BM / 4)) * 4, k = e / (BM / 4);
          *reinterpret_cast<float4*>(&As[k][m]) = make_float4(ra[4 * i], ra[4 * i + 1], ra[4 * i + 2], ra[4 * i + 3]);
        } else {
          const int k = (e & 3) * 4, m = e >> 2;
#pragma unroll
          for (int u = 0; u < 4; ++u) As[k + u][m] = ra[4 * i + u];
        }
      }
#pragma unroll
      for (int i = 0; i < VB; ++i) {
        const int e = tid + i * 256;
        if (e < BN * BK / 4) {
          if (TRB) {
            const int k = (e & 3) * 4, n = e >> 2;
#pragma unroll
            for (int u = 0; u < 4; ++u) Bs[k + u][n] = rb[4 * i + u];
          } else {
            const int n = (e % (BN / 4)) * 4, k = e / (BN / 4);
            *reinterpret_cast<float4*>(&Bs[k][n]) = make_float4(rb[4 * i], rb[4 * i + 1], rb[4 * i + 2], rb[4 * i + 3]);
          }
        }
      }
      return;
    }
#pragma unroll
    for (int i = 0; i < LA; ++i) {
      const int e = tid + i * 256;
      if (TRA) As[e / BM][e % BM] = ra[i];
      else As[e & 15][e >> 4] = ra[i];
    }
#pragma unroll
    for (int i = 0; i < LB; ++i) {
      const int e = tid + i * 256;
      if (TRB) Bs[e & 15][e >> 4] = rb[i];
      else Bs[e / BN][e % BN] = rb[i];
    }
  };

  fetch(0);
  for (int k0 = 0; k0 < Kend; k0 += BK) {
    stash();
    __syncthreads();
    if (k0 + BK < Kend) fetch(k0 + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float4 av[RM];
#pragma unroll
      for (int g = 0; g < RM; ++g) av[g] = *reinterpret_cast<const float4*>(&As[kk][g * 64 + ty * 4]);
      float bb[CN];
      if (CN == 4) {
        const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
        bb[0] = bv.x; bb[1] = bv.y; bb[2] = bv.z; bb[CN - 1] = bv.w;
      } else {
#pragma unroll
        for (int j = 0; j < CN; ++j) bb[j] = Bs[kk][tx * CN + j];
      }
#pragma unroll
      for (int g = 0; g < RM; ++g) {
        const float a[4] = {av[g].x, av[g].y, av[g].z, av[g].w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < CN; ++j) acc[g * 4 + i][j] = fmaf(a[i], bb[j], acc[g * 4 + i][j]);
      }
    }
    __syncthreads();
  }
  // symmetric output: a tile writes its entries on or above the diagonal and their mirror
  // images, so each pair is produced exactly once and C is symmetric bit for bit
  const bool sym = (flags & GEMM_SYM) != 0;
#pragma unroll
  for (int g = 0; g < RM; ++g)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int gm = m0 + g * 64 + ty * 4 + i;
      if (gm >= M) continue;
#pragma unroll
      for (int j = 0; j < CN; ++j) {
        const int gn = n0 + tx * CN + j;
        if (gn < N && (!sym || gn >= gm)) {
          C[(size_t)gm * ldc + gn] = acc[g * 4 + i][j];
          if (sym && gn > gm) C[(size_t)gn * ldc + gm] = acc[g * 4 + i][j];
        }
      }
    }
}

template <typename TA, typename TB, bool TRA, bool TRB, int RM, int CN>
static void gemm_launch(const TA* A, const TB* B, float* C, int M, int N, int K, int lda, int ldb,
                        int ldc, size_t sA, size_t sB, size_t sC, int batch, cudaStream_t st,
                        int flags) {
  dim3 grid((N + 16 * CN - 1) / (16 * CN), (M + 64 * RM - 1) / (64 * RM), batch);
  { gemm_kernel<TA, TB, TRA, TRB, RM, CN><<<grid, 256, 0, st>>>(A, B, C, M, N, K, lda, ldb, ldc, sA, sB, sC, flags); note_launch(); }
}

// ==========================================================================================
// The same product for float32 operands whose output is 48 k columns wide (the subspace
// dimension 144 = 3 * 48):  C[m][n] = sum_k A[m][k] * opB[k][n],  A row-major.
// (64 RM) x 48 tile per block of 192 threads = 12 (columns, four each) x 16 (rows, four in each
// of RM groups of 64): a 16-deep slice costs RM + 1 16-byte reads of shared memory per 16 RM
// multiply-adds, against RM + 3 reads per 12 RM in the kernel above.  Needs every operand
// address 16-byte aligned (the caller checks).
// ==========================================================================================
template <bool TRB, int RM>
__global__ void __launch_bounds__(192, 2) gemm_tall_kernel(const float* __restrict__ A,
                                                          const float* __restrict__ B,
                                                          float* __restrict__ C, int M, int N, int K,
                                                          int lda, int ldb, int ldc, size_t sA,
                                                          size_t sB, size_t sC, int flags) {
  constexpr int BM = 64 * RM, BN = 48, BK = 16;
  constexpr int NVA = BM * BK / 4, VA = (NVA + 191) / 192;  // A vectors per slice, per thread
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  A += (size_t)blockIdx.z * sA;
  B += (size_t)blockIdx.z * sB;
  C += (size_t)blockIdx.z * sC;
  const int tid = threadIdx.x, tx = tid % 12, ty = tid / 12;
  const int Kend = (flags & GEMM_B_UPPER) ? min(K, n0 + BN) : K;
  float acc[4 * RM][4];
#pragma unroll
  for (int i = 0; i < 4 * RM; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  float4 ra[VA], rb;
  auto fetch = [&](int k0) {
#pragma unroll
    for (int i = 0; i < VA; ++i) {
      const int e = tid + i * 192;
      const int k = (e & 3) * 4, m = e >> 2;  // stored [m][k]: vectors run along k
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (e < NVA && m0 + m < M && k0 + k < Kend)
        v = __ldg(reinterpret_cast<const float4*>(A + (size_t)(m0 + m) * lda + k0 + k));
      ra[i] = v;
    }
    {
      int n, k;
      if (TRB) {  // stored [n][k]: vectors run along k
        k = (tid & 3) * 4;
        n = tid >> 2;
      } else {  // stored [k][n]: vectors run along n
        n = (tid % 12) * 4;
        k = tid / 12;
      }
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (n0 + n < N && k0 + k < Kend)
        v = __ldg(reinterpret_cast<const float4*>(
            TRB ? B + (size_t)(n0 + n) * ldb + k0 + k : B + (size_t)(k0 + k) * ldb + n0 + n));
      rb = v;
    }
  };
  auto stash = [&]() {
#pragma unroll
    for (int i = 0; i < VA; ++i) {
      const int e = tid + i * 192;
      if (e < NVA) {
        const int k = (e & 3) * 4, m = e >> 2;
        As[k][m] = ra[i].x;
        As[k + 1][m] = ra[i].y;
        As[k + 2][m] = ra[i].z;
        As[k + 3][m] = ra[i].w;
      }
    }
    if (TRB) {
      const int k = (tid & 3) * 4, n = tid >> 2;
      Bs[k][n] = rb.x;
      Bs[k + 1][n] = rb.y;
      Bs[k + 2][n] = rb.z;
      Bs[k + 3][n] = rb.w;
    } else {
      *reinterpret_cast<float4*>(&Bs[tid / 12][(tid % 12) * 4]) = rb;
    }
  };
  fetch(0);
  for (int k0 = 0; k0 < Kend; k0 += BK) {
    stash();
    __syncthreads();
    if (k0 + BK < Kend) fetch(k0 + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float bb[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int g = 0; g < RM; ++g) {
        const float4 av = *reinterpret_cast<const float4*>(&As[kk][g * 64 + ty * 4]);
        const float a[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[g * 4 + i][j] = fmaf(a[i], bb[j], acc[g * 4 + i][j]);
      }
    }
    __syncthreads();
  }
  const int gn = n0 + tx * 4;
  if (gn >= N) return;  // N is a multiple of four: a thread's four columns are in or out together
#pragma unroll
  for (int g = 0; g < RM; ++g)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int gm = m0 + g * 64 + ty * 4 + i;
      if (gm < M)
        *reinterpret_cast<float4*>(C + (size_t)gm * ldc + gn) =
            make_float4(acc[g * 4 + i][0], acc[g * 4 + i][1], acc[g * 4 + i][2], acc[g * 4 + i][3]);
    }
}

// The same tile for opB = B (stored [k][n]), the product with the long inner dimension (G Q):
// both operands keep their global layout in shared memory, so slices arrive by asynchronous
// 16-byte copies, TALL_STAGES of them in flight, with one barrier per slice.  A is held as
// [m][16] with the four vectors of a row permuted by (m / 4) mod 4, which spreads the rows a
// warp reads at once over the banks.
constexpr int TALL_STAGES = 4;

template <int RM>
__global__ void __launch_bounds__(192, 2) gemm_tall_nn_kernel(const float* __restrict__ A,
                                                             const float* __restrict__ B,
                                                             float* __restrict__ C, int M, int N, int K,
                                                             int lda, int ldb, int ldc, size_t sA,
                                                             size_t sB, size_t sC) {
  constexpr int BM = 64 * RM, BN = 48, BK = 16;
  constexpr int ATILE = BM * BK, STAGE = ATILE + BK * BN;
  extern __shared__ __align__(16) float tall_smem[];  // [stage][A: BM x 16 | B: 16 x 48]
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  A += (size_t)blockIdx.z * sA;
  B += (size_t)blockIdx.z * sB;
  C += (size_t)blockIdx.z * sC;
  const int tid = threadIdx.x, tx = tid % 12, ty = tid / 12;
  const int nslice = (K + BK - 1) / BK;
  float acc[4 * RM][4];
#pragma unroll
  for (int i = 0; i < 4 * RM; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  auto issue = [&](int slice) {
    if (slice < nslice) {
      float* st = tall_smem + (slice % TALL_STAGES) * STAGE;
      const int k0 = slice * BK;
#pragma unroll
      for (int i = 0; i < (BM * 4 + 191) / 192; ++i) {
        const int e = tid + i * 192;  // vector e: row m = e / 4, vector c = e % 4 of the row
        if (e < BM * 4) {
          const int m = e >> 2, c = e & 3;
          const bool ok = (m0 + m < M) && (k0 + c * 4 < K);
          const float* src = ok ? A + (size_t)(m0 + m) * lda + k0 + c * 4 : A;
          cp_async16(st + m * BK + ((c ^ ((m >> 2) & 3)) << 2), src, ok ? 16 : 0);
        }
      }
      {
        const int kr = tid / 12, cvn = (tid % 12) * 4;
        const bool ok = (k0 + kr < K) && (n0 + cvn < N);
        const float* src = ok ? B + (size_t)(k0 + kr) * ldb + n0 + cvn : B;
        cp_async16(st + ATILE + kr * BN + cvn, src, ok ? 16 : 0);
      }
    }
    cp_async_commit();
  };
#pragma unroll
  for (int p = 0; p < TALL_STAGES - 1; ++p) issue(p);
  const int sw = ty & 3;
  for (int slice = 0; slice < nslice; ++slice) {
    cp_async_wait<TALL_STAGES - 2>();
    __syncthreads();
    issue(slice + TALL_STAGES - 1);
    const float* As = tall_smem + (slice % TALL_STAGES) * STAGE;
    const float* Bs = As + ATILE;
#pragma unroll
    for (int k4 = 0; k4 < 4; ++k4) {
      float4 bv[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) bv[u] = *reinterpret_cast<const float4*>(Bs + (k4 * 4 + u) * BN + tx * 4);
#pragma unroll
      for (int g = 0; g < RM; ++g)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float4 av = *reinterpret_cast<const float4*>(As + (g * 64 + ty * 4 + i) * BK + ((k4 ^ sw) << 2));
          const float a[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            acc[g * 4 + i][0] = fmaf(a[u], bv[u].x, acc[g * 4 + i][0]);
            acc[g * 4 + i][1] = fmaf(a[u], bv[u].y, acc[g * 4 + i][1]);
            acc[g * 4 + i][2] = fmaf(a[u], bv[u].z, acc[g * 4 + i][2]);
            acc[g * 4 + i][3] = fmaf(a[u], bv[u].w, acc[g * 4 + i][3]);
          }
        }
    }
  }
  cp_async_wait<0>();
  const int gn = n0 + tx * 4;
  if (gn >= N) return;
#pragma unroll
  for (int g = 0; g < RM; ++g)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int gm = m0 + g * 64 + ty * 4 + i;
      if (gm < M)
        *reinterpret_cast<float4*>(C + (size_t)gm * ldc + gn) =
            make_float4(acc[g * 4 + i][0], acc[g * 4 + i][1], acc[g * 4 + i][2], acc[g * 4 + i][3]);
    }
}

template <bool TRB>
static bool gemm_tall(const float* A, const float* B, float* C, int M, int N, int K, int lda, int ldb,
                      int ldc, size_t sA, size_t sB, size_t sC, int batch, cudaStream_t st, int flags) {
  if (N % 48 != 0 || M < 128 && M != 144 || ((lda | ldb | ldc | K) & 3) != 0 ||
      ((sA | sB | sC) & 3) != 0 || ((((uintptr_t)A) | ((uintptr_t)B) | ((uintptr_t)C)) & 15) != 0)
    return false;
  // rows per tile: 192 unless 128 wastes less of the last tile
  const bool three = ((M + 191) / 192) * 192 <= ((M + 127) / 128) * 128;
  if (three) {
    dim3 grid(N / 48, (M + 191) / 192, batch);
    if (!TRB && !(flags & GEMM_B_UPPER)) {
      const size_t smem = (size_t)TALL_STAGES * (192 * 16 + 16 * 48) * sizeof(float);
      cudaFuncSetAttribute((const void*)gemm_tall_nn_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      { gemm_tall_nn_kernel<3><<<grid, 192, smem, st>>>(A, B, C, M, N, K, lda, ldb, ldc, sA, sB, sC); note_launch(); }
      return true;
    }
    { gemm_tall_kernel<TRB, 3><<<grid, 192, 0, st>>>(A, B, C, M, N, K, lda, ldb, ldc, sA, sB, sC, flags); note_launch(); }
  } else {
    dim3 grid(N / 48, (M + 127) / 128, batch);
    { gemm_tall_kernel<TRB, 2><<<grid, 192, 0, st>>>(A, B, C, M, N, K, lda, ldb, ldc, sA, sB, sC, flags); note_launch(); }
  }
  return true;
}

template <typename TA, typename TB, bool TRA, bool TRB>
static void gemm(const TA* A, const TB* B, float* C, int M, int N, int K, int lda, int ldb,
                 int ldc, size_t sA, size_t sB, size_t sC, int batch, cudaStream_t st,
                 int cls = KC_GEMM, int flags = 0) {
  Scope scope_(cls, st);
  if constexpr (std::is_same<TA, float>::value && std::is_same<TB, float>::value && !TRA) {
    if (!(flags & GEMM_SYM) &&
        gemm_tall<TRB>(A, B, C, M, N, K, lda, ldb, ldc, sA, sB, sC, batch, st, flags))
      return;
  }
  // column tiles of 48 when they pad the width less than tiles of 64 (e.g. 144 = 3 * 48)
  const bool narrow = ((N + 47) / 48) * 48 < ((N + 63) / 64) * 64;
  if (M >= 256 && !(flags & GEMM_SYM)) {
    if (narrow) gemm_launch<TA, TB, TRA, TRB, 2, 3>(A, B, C, M, N, K, lda, ldb, ldc, sA, sB, sC, batch, st, flags);
    else gemm_launch<TA, TB, TRA, TRB, 2, 4>(A, B, C, M, N, K, lda, ldb, ldc, sA, sB, sC, batch, st, flags);
  } else {
    if (narrow) gemm_launch<TA, TB, TRA, TRB, 1, 3>(A, B, C, M, N, K, lda, ldb, ldc, sA, sB, sC, batch, st, flags);
    else gemm_launch<TA, TB, TRA, TRB, 1, 4>(A, B, C, M, N, K, lda, ldb, ldc, sA, sB, sC, batch, st, flags);
  }
}

// ==========================================================================================
// C = A^T B for tall operands with few columns (n <= 144, n a multiple of 4), where C is known
// to be symmetric (A = B, or B = G A with G symmetric): only the entries on or above the
// diagonal are computed and each is written to both places.
//   A, B [K][n] row-major;  C parts: [nparts][n][n] per image, part s = the sum over the s-th
//   chunk of K.  The consumer adds the parts (in order, so the result is deterministic).
// One block per (chunk, image): 192 threads.  The columns are split in a low and a high half;
// thread (ty, tx), tx >= ty, of the triangular grid holds rows {4 ty.., half + 4 ty..} x columns
// {4 tx.., half + 4 tx..}: four 4 x 4 blocks, of which three lie on or above the diagonal and the
// fourth is the mirror image of a block no thread of the triangle holds.  A 16-deep slice costs
// four 16-byte reads of shared memory (neighbouring threads read neighbouring vectors) per 64
// multiply-adds.
// ==========================================================================================
constexpr int TN_MAX = 144, TN_LD = 152, TN_PARTS = 4;

constexpr int TN_STAGES = 4;  // slices in flight (asynchronous copies straight into shared memory)

template <bool SAME>
__global__ void __launch_bounds__(192) gemm_tn_upper_kernel(const float* __restrict__ A,
                                                           const float* __restrict__ B,
                                                           float* __restrict__ C, int n, int K,
                                                           int chunk, size_t sA, size_t sB,
                                                           size_t sC) {
  extern __shared__ __align__(16) float tn_smem[];  // [stage][A, B][16][TN_LD]
  constexpr int TILE = 16 * TN_LD, STAGE = (SAME ? 1 : 2) * TILE;
  const int tid = threadIdx.x, s = blockIdx.x, img = blockIdx.y;
  A += (size_t)img * sA;
  B += (size_t)img * sB;
  C += (size_t)img * sC + (size_t)s * n * n;
  const int k_lo = s * chunk, k_hi = min(K, k_lo + chunk);
  const int nslice = (k_hi > k_lo) ? (k_hi - k_lo + 15) >> 4 : 0;
  const int nt = (n + 7) >> 3;  // tiles per side; the high half starts at column 4 nt
  const int half = 4 * nt;
  int ty = 0, rem = tid;
  while (ty < nt && rem >= nt - ty) {
    rem -= nt - ty;
    ++ty;
  }
  const bool active = ty < nt;
  const int tx = ty + rem;
  const int nv = n >> 2;                 // 16-byte vectors per row
  const int nvec = 16 * nv;              // per slice
  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
  // this thread's (at most three) vectors of a slice: row kr[i] of the slice, vector cv[i]
  int kr[3], cv[3];
#pragma unroll
  for (int i = 0; i < 3; ++i) {
    const int e = tid + i * 192;
    kr[i] = (e < nvec) ? e / nv : -1;
    cv[i] = (e < nvec) ? e - kr[i] * nv : 0;
  }
  auto issue = [&](int slice) {
    if (slice < nslice) {
      float* st = tn_smem + (slice % TN_STAGES) * STAGE;
      const int k0 = k_lo + slice * 16;
#pragma unroll
      for (int i = 0; i < 3; ++i) {
        if (kr[i] < 0) continue;
        const bool ok = k0 + kr[i] < k_hi;
        const size_t off = (size_t)(ok ? k0 + kr[i] : k_lo) * n + cv[i] * 4;
        cp_async16(st + kr[i] * TN_LD + cv[i] * 4, A + off, ok ? 16 : 0);
        if (!SAME) cp_async16(st + TILE + kr[i] * TN_LD + cv[i] * 4, B + off, ok ? 16 : 0);
      }
    }
    cp_async_commit();  // (an empty group keeps the count of groups in step with the slices)
  };
#pragma unroll
  for (int p = 0; p < TN_STAGES - 1; ++p) issue(p);
  for (int slice = 0; slice < nslice; ++slice) {
    cp_async_wait<TN_STAGES - 2>();  // this thread's copies of `slice` have landed
    __syncthreads();                 // everyone's have, and everyone is done with slice - 1
    issue(slice + TN_STAGES - 1);    // into the buffer slice - 1 used
    if (active) {
      const float* As = tn_smem + (slice % TN_STAGES) * STAGE;
      const float* Bt = SAME ? As : As + TILE;
      // the operands of step kk + 1 are read before the multiply-adds of step kk are issued
      float4 na0 = *reinterpret_cast<const float4*>(As + ty * 4);
      float4 na1 = *reinterpret_cast<const float4*>(As + half + ty * 4);
      float4 nb0 = *reinterpret_cast<const float4*>(Bt + tx * 4);
      float4 nb1 = *reinterpret_cast<const float4*>(Bt + half + tx * 4);
#pragma unroll
      for (int kk = 0; kk < 16; ++kk) {
        const float4 a0 = na0, a1 = na1, b0 = nb0, b1 = nb1;
        if (kk + 1 < 16) {
          na0 = *reinterpret_cast<const float4*>(As + (kk + 1) * TN_LD + ty * 4);
          na1 = *reinterpret_cast<const float4*>(As + (kk + 1) * TN_LD + half + ty * 4);
          nb0 = *reinterpret_cast<const float4*>(Bt + (kk + 1) * TN_LD + tx * 4);
          nb1 = *reinterpret_cast<const float4*>(Bt + (kk + 1) * TN_LD + half + tx * 4);
        }
        const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
        const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
      }
    }
  }
  cp_async_wait<0>();
  if (!active) return;
  // every unordered pair {r, c} is produced by exactly one thread and written to both places
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = (i < 4) ? ty * 4 + i : half + ty * 4 + i - 4;
    if (r >= n) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int c = (j < 4) ? tx * 4 + j : half + tx * 4 + j - 4;
      if (c >= n) continue;
      if (c >= r || tx > ty) {
        C[(size_t)r * n + c] = acc[i][j];
        if (c != r) C[(size_t)c * n + r] = acc[i][j];
      }
    }
  }
}

// Number of parts the k x k products A^T B are delivered in (1 = the general kernel).
int tn_parts(int k) { return (k <= TN_MAX && (k & 3) == 0 && k >= 8) ? TN_PARTS : 1; }

// C (nparts parts per image, image stride nparts * n * n) = A^T B, symmetric.
static void gemm_tn_sym(const float* A, const float* B, float* C, int n, int K, size_t sA, size_t sB,
                        int batch, cudaStream_t st, int cls) {
  const int parts = tn_parts(n);
  if (parts == 1) {
    gemm<float, float, true, false>(A, B, C, n, n, K, n, n, n, sA, sB, (size_t)n * n, batch, st, cls,
                                    A == B ? GEMM_SYM : 0);
    return;
  }
  Scope scope_(cls, st);
  const int chunk = ((K + parts - 1) / parts + 15) / 16 * 16;
  dim3 grid(parts, batch);
  const size_t sC = (size_t)parts * n * n;
  if (A == B) {
    const size_t smem = (size_t)TN_STAGES * 16 * TN_LD * sizeof(float);
    cudaFuncSetAttribute((const void*)gemm_tn_upper_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    { gemm_tn_upper_kernel<true><<<grid, 192, smem, st>>>(A, B, C, n, K, chunk, sA, sB, sC); note_launch(); }
  } else {
    const size_t smem = (size_t)TN_STAGES * 2 * 16 * TN_LD * sizeof(float);
    cudaFuncSetAttribute((const void*)gemm_tn_upper_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    { gemm_tn_upper_kernel<false><<<grid, 192, smem, st>>>(A, B, C, n, K, chunk, sA, sB, sC); note_launch(); }
  }
}

// G = O O^T for float32 inputs (and, until the tensor-core kernel takes over, float16 ones).
tc_status launch_gram_simt(const Dims& D, const void* O, float* G, cudaStream_t st) {
  const size_t sO = (size_t)D.N * D.d, sG = (size_t)D.N * D.N;
  TC_WITH_STORAGE_TYPE(D,
    gemm<T, T, false, true>((const T*)O, (const T*)O, G, D.N, D.N, D.d, D.d, D.d, D.N, sO, sO, sG, D.B,
                            st, KC_GRAM););
  return TC_OK;
}

// ==========================================================================================
// Sign sketch of O:  Y[x][j] = sum over columns c == j (mod k) of s(c) O[x][c],  s(c) = +-1
// from a fixed integer hash.  grid (N, B), block k.  It only has to capture the dominant
// column space of O; the steps after it correct it against G itself.
// ==========================================================================================
__device__ inline float hash_sign(uint32_t c) {
  uint32_t h = c * 2654435761u;
  h ^= h >> 15;
  h *= 2246822519u;
  h ^= h >> 13;
  return (h & 1u) ? 1.f : -1.f;
}

template <typename T>
__global__ void sketch_kernel(const T* __restrict__ O, float* __restrict__ Y, int N, int d, int k) {
  const int x = blockIdx.x, b = blockIdx.y, j = threadIdx.x;
  if (j >= k) return;
  const T* row = O + ((size_t)b * N + x) * d;
  float acc = 0.f;
  for (int c = j; c < d; c += k) acc += hash_sign((uint32_t)c) * ld_f32(row + c);
  Y[((size_t)b * N + x) * k + j] = acc;
}

// The same sketch with 16-byte loads, for k a multiple of the vector length L (8 halves or 4
// floats): columns are taken in groups of L, group g goes to bucket group g mod (k / L), column
// i of the group to bucket i of that bucket group.  block (k / L, rows), grid (N / rows, B).
template <typename T, int L>
__global__ void sketch_vec_kernel(const T* __restrict__ O, float* __restrict__ Y, int N, int d, int k) {
  extern __shared__ float sgn[];  // [d]
  const int kg = blockDim.x, tx = threadIdx.x, ty = threadIdx.y;
  const int b = blockIdx.y, x = blockIdx.x * blockDim.y + ty;
  for (int c = ty * kg + tx; c < d; c += kg * blockDim.y) sgn[c] = hash_sign((uint32_t)c);
  __syncthreads();
  if (x >= N) return;
  const uint4* row = reinterpret_cast<const uint4*>(O + ((size_t)b * N + x) * d);
  const int ng = d / L;
  float acc[L];
#pragma unroll
  for (int i = 0; i < L; ++i) acc[i] = 0.f;
  int g = tx;
  for (; g + 7 * kg < ng; g += 8 * kg) {  // eight 16-byte loads in flight per thread
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = __ldg(row + g + u * kg);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const T* e = reinterpret_cast<const T*>(&v[u]);
      const float* sg = sgn + (size_t)(g + u * kg) * L;
#pragma unroll
      for (int i = 0; i < L; ++i) acc[i] = fmaf(sg[i], (float)e[i], acc[i]);
    }
  }
  for (; g < ng; g += kg) {
    const uint4 v = __ldg(row + g);
    const T* e = reinterpret_cast<const T*>(&v);
    const float* sg = sgn + (size_t)g * L;
#pragma unroll
    for (int i = 0; i < L; ++i) acc[i] = fmaf(sg[i], (float)e[i], acc[i]);
  }
  float* out = Y + ((size_t)b * N + x) * k + tx * L;
#pragma unroll
  for (int i = 0; i < L; ++i) out[i] = acc[i];
}

// ==========================================================================================
// Cholesky factor of S (+ shift) and its inverse.  One block per image.
//   S [k][k] symmetric in;  RinvT [k][k] out, RinvT[c][m] = (R^{-1})[m][c] for m <= c, else 0,
//   where R^T R = S + shift_rel * max_i S_ii * I.  Then  Y R^{-1}  has (nearly) orthonormal
//   columns: one pass of Cholesky-QR.  The shift keeps the factorisation alive when S is
//   numerically singular; a later unshifted pass removes its effect.
// The k x k work arrays live in shared memory when they fit, else in global memory.
// ==========================================================================================
__global__ void __launch_bounds__(512) chol_inv_kernel(const float* __restrict__ S,
                                                      float* __restrict__ RinvT,
                                                      float* __restrict__ Rwork, int k,
                                                      float shift_rel, int use_smem,
                                                      int32_t* __restrict__ status) {
  extern __shared__ float sm[];
  __shared__ float s_red[16];
  __shared__ float s_piv;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t kk = (size_t)k * k;
  const float* Sb = S + b * kk;
  float* R = use_smem ? sm : Rwork + b * kk;        // upper triangle used
  float* XT = use_smem ? sm + kk : RinvT + b * kk;  // XT[c][m]
  float* out = RinvT + b * kk;

  float md = 0.f;
  for (int i = tid; i < k; i += 512) md = fmaxf(md, Sb[(size_t)i * k + i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) md = fmaxf(md, __shfl_xor_sync(0xffffffffu, md, o));
  if (lane == 0) s_red[warp] = md;
  __syncthreads();
  md = s_red[0];
  for (int w = 1; w < 16; ++w) md = fmaxf(md, s_red[w]);
  const float shift = shift_rel * md;
  for (size_t e = tid; e < kk; e += 512) {
    const int r = (int)(e / k), c = (int)(e % k);
    float v = Sb[e];
    if (r == c) v += shift;
    R[e] = v;
  }
  __syncthreads();

  bool bad = false;
  for (int j = 0; j < k; ++j) {
    if (tid == 0) {
      float p = R[(size_t)j * k + j];
      if (!(p > 0.f)) {
        p = fmaxf(md, 1e-30f) * 1e-12f;
        bad = true;
      }
      s_piv = sqrtf(p);
    }
    __syncthreads();
    const float dj = s_piv, inv = 1.0f / dj;
    for (int c = j + tid; c < k; c += 512) R[(size_t)j * k + c] = (c == j) ? dj : R[(size_t)j * k + c] * inv;
    __syncthreads();
    for (int r = j + 1 + warp; r < k; r += 16) {
      const float f = R[(size_t)j * k + r];
      for (int c = r + lane; c < k; c += 32) R[(size_t)r * k + c] = fmaf(-f, R[(size_t)j * k + c], R[(size_t)r * k + c]);
    }
    __syncthreads();
  }
  if (tid == 0 && bad) atomicMax(&status[b], (int)TC_ERR_BREAKDOWN);

  // inverse, one warp per column c of R^{-1}:  R x = e_c by back substitution
  for (int c = warp; c < k; c += 16) {
    float* x = XT + (size_t)c * k;
    if (lane == 0) x[c] = 1.0f / R[(size_t)c * k + c];
    __syncwarp();
    for (int i = c - 1; i >= 0; --i) {
      float s = 0.f;
      for (int m = i + 1 + lane; m <= c; m += 32) s = fmaf(R[(size_t)i * k + m], x[m], s);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) x[i] = -s / R[(size_t)i * k + i];
      __syncwarp();
    }
    for (int m = c + 1 + lane; m < k; m += 32) x[m] = 0.f;
  }
  __syncthreads();
  if (use_smem)
    for (size_t e = tid; e < kk; e += 512) out[e] = XT[e];
}

// ==========================================================================================
// The same factorisation and inverse for k small enough that one k x k float32 array fits in
// shared memory: blocked (16 columns at a time) so that the block-wide barriers number a few
// dozen instead of three per column, and the inverse is formed in place of the factor.
//   phase 1  R^T R = S + shift I   (right-looking: diagonal block in one warp's registers,
//            block row by forward substitution, trailing update in 4 x 4 register tiles)
//   phase 2  R <- R^{-1}           (left to right over block columns; a finished leading
//            block of the inverse multiplies the next block column)
// ==========================================================================================
constexpr int CNB = 16;

__global__ void __launch_bounds__(512) chol_inv_blocked_kernel(const float* __restrict__ S,
                                                              float* __restrict__ RinvT, int k,
                                                              float shift_rel,
                                                              int32_t* __restrict__ status,
                                                              int nparts) {
  extern __shared__ float A[];  // [k][ld], ld odd: rows and columns both walk all banks
  __shared__ float s_red[16];
  __shared__ float s_row[2][CNB];
  __shared__ int s_bad;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ld = k | 1;
  const size_t kk = (size_t)k * k;
  const float* Sb = S + (size_t)b * nparts * kk;  // S arrives as nparts parts to be added up

  float md = 0.f;
  for (int i = tid; i < k; i += 512) {
    float dsum = 0.f;
    for (int q = 0; q < nparts; ++q) dsum += __ldg(Sb + q * kk + (size_t)i * k + i);
    md = fmaxf(md, dsum);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) md = fmaxf(md, __shfl_xor_sync(0xffffffffu, md, o));
  if (lane == 0) s_red[warp] = md;
  if (tid == 0) s_bad = 0;
  __syncthreads();
  md = s_red[0];
  for (int w = 1; w < 16; ++w) md = fmaxf(md, s_red[w]);
  const float shift = shift_rel * md;
  const float tiny = fmaxf(md, 1e-30f) * 1e-12f;
  if (nparts == 4 && (k & 3) == 0) {
    // four parts, sixteen bytes at a time: all the loads of a trip are in flight together
    const float4* S4 = reinterpret_cast<const float4*>(Sb);
    const int kv = k >> 2, nv = (int)(kk >> 2);
    for (int e = tid; e < nv; e += 512) {
      const float4 p0 = __ldg(S4 + e), p1 = __ldg(S4 + nv + e), p2 = __ldg(S4 + 2 * nv + e),
                   p3 = __ldg(S4 + 3 * nv + e);
      const int r = e / kv, c = (e - r * kv) * 4;
      float* dst = A + r * ld + c;
      dst[0] = ((p0.x + p1.x) + (p2.x + p3.x)) + (r == c ? shift : 0.f);
      dst[1] = ((p0.y + p1.y) + (p2.y + p3.y)) + (r == c + 1 ? shift : 0.f);
      dst[2] = ((p0.z + p1.z) + (p2.z + p3.z)) + (r == c + 2 ? shift : 0.f);
      dst[3] = ((p0.w + p1.w) + (p2.w + p3.w)) + (r == c + 3 ? shift : 0.f);
    }
  } else {
    for (int e = tid; e < (int)kk; e += 512) {
      const int r = e / k, c = e - r * k;
      float v = 0.f;
      for (int q = 0; q < nparts; ++q) v += Sb[q * kk + e];
      A[r * ld + c] = v + (r == c ? shift : 0.f);
    }
  }
  __syncthreads();

  const int nblk = (k + CNB - 1) / CNB;
  // ---------------- phase 1: Cholesky ----------------
  for (int jb = 0; jb < nblk; ++jb) {
    const int j0 = jb * CNB, j1 = min(k, j0 + CNB);
    if (warp == 0) {
      // lane c (< 16) keeps column c of the diagonal block; rows/columns past k act as identity
      float col[CNB];
      const int gc = j0 + lane;
#pragma unroll
      for (int r = 0; r < CNB; ++r) {
        const int gr = j0 + r;
        float v = (r == lane) ? 1.f : 0.f;
        if (lane < CNB && gc < k && gr < k && r <= lane) v = A[gr * ld + gc];
        col[r] = v;
      }
#pragma unroll
      for (int i = 0; i < CNB; ++i) {
        float piv = __shfl_sync(0xffffffffu, col[i], i);
        if (!(piv > 0.f)) {
          piv = tiny;
          if (lane == 0) s_bad = 1;
        }
        const float rinv = rsqrtf(piv);
        if (lane == i) col[i] = piv * rinv;
        else if (lane > i) col[i] = col[i] * rinv;
        // row i of the factor goes through shared memory: broadcast reads pipeline, a chain
        // of fifteen shuffles does not
        if (lane < CNB) s_row[i & 1][lane] = col[i];
        __syncwarp();
#pragma unroll
        for (int r = i + 1; r < CNB; ++r) {
          const float v = s_row[i & 1][r];
          if (lane >= r) col[r] = fmaf(-v, col[i], col[r]);
        }
      }
#pragma unroll
      for (int r = 0; r < CNB; ++r) {
        const int gr = j0 + r;
        if (lane < CNB && gc < k && gr < k && r <= lane) A[gr * ld + gc] = col[r];
      }
    }
    __syncthreads();
    // block row: R[j0.., c] for c >= j1, one thread per column
    for (int c = j1 + tid; c < k; c += 512) {
      float x[CNB];
#pragma unroll
      for (int i = 0; i < CNB; ++i) {
        if (j0 + i < k) {
          float sacc = A[(j0 + i) * ld + c];
#pragma unroll
          for (int m = 0; m < i; ++m) sacc = fmaf(-A[(j0 + m) * ld + j0 + i], x[m], sacc);
          x[i] = sacc / A[(j0 + i) * ld + j0 + i];
        } else {
          x[i] = 0.f;
        }
      }
#pragma unroll
      for (int i = 0; i < CNB; ++i)
        if (j0 + i < k) A[(j0 + i) * ld + c] = x[i];
    }
    __syncthreads();
    // trailing update of the upper triangle in 4 x 4 tiles
    const int m = k - j1;
    if (m > 0) {
      const int mt = (m + 3) >> 2;
      for (int t = tid; t < mt * mt; t += 512) {
        const int tr = t / mt, tc = t - tr * mt;
        if (tc < tr) continue;
        const int r0 = j1 + 4 * tr, c0 = j1 + 4 * tc;
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 4
        for (int i = j0; i < j1; ++i) {
          float a[4], bb[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            a[u] = (r0 + u < k) ? A[i * ld + r0 + u] : 0.f;
            bb[u] = (c0 + u < k) ? A[i * ld + c0 + u] : 0.f;
          }
#pragma unroll
          for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(a[u], bb[v], acc[u][v]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
          for (int v = 0; v < 4; ++v)
            if (r0 + u < k && c0 + v < k && c0 + v >= r0 + u) A[(r0 + u) * ld + c0 + v] -= acc[u][v];
      }
    }
    __syncthreads();
  }
  if (tid == 0 && s_bad) atomicMax(&status[b], (int)TC_ERR_BREAKDOWN);

  // ---------------- phase 2: in-place inverse of the upper-triangular factor ----------------
  for (int jb = 0; jb < nblk; ++jb) {
    const int j0 = jb * CNB, j1 = min(k, j0 + CNB), w = j1 - j0;
    if (warp == 0) {
      // lane c solves R_JJ x = e_c by back substitution (x has entries 0..c)
      float x[CNB];
#pragma unroll
      for (int i = 0; i < CNB; ++i) x[i] = 0.f;
      if (lane < w) {
#pragma unroll
        for (int i = CNB - 1; i >= 0; --i) {
          if (i <= lane) {
            float sacc = (i == lane) ? 1.f : 0.f;
#pragma unroll
            for (int mm = i + 1; mm < CNB; ++mm)
              if (mm <= lane) sacc = fmaf(-A[(j0 + i) * ld + j0 + mm], x[mm], sacc);
            x[i] = sacc / A[(j0 + i) * ld + j0 + i];
          }
        }
      }
      __syncwarp();
      if (lane < w) {
#pragma unroll
        for (int i = 0; i < CNB; ++i)
          if (i <= lane) A[(j0 + i) * ld + j0 + lane] = x[i];
      }
    }
    __syncthreads();
    if (j0 > 0) {
      // T = R[0:j0, J] * X_JJ, one thread per row, written back over R[0:j0, J]
      for (int r = tid; r < j0; r += 512) {
        float rr[CNB], tt[CNB];
#pragma unroll
        for (int mm = 0; mm < CNB; ++mm) rr[mm] = (mm < w) ? A[r * ld + j0 + mm] : 0.f;
#pragma unroll
        for (int c = 0; c < CNB; ++c) {
          float sacc = 0.f;
#pragma unroll
          for (int mm = 0; mm <= c; ++mm)
            if (c < w) sacc = fmaf(rr[mm], A[(j0 + mm) * ld + j0 + c], sacc);
          tt[c] = sacc;
        }
#pragma unroll
        for (int c = 0; c < CNB; ++c)
          if (c < w) A[r * ld + j0 + c] = tt[c];
      }
      __syncthreads();
      // X[0:j0, J] = - X[0:j0, 0:j0] * T.  A thread owns one row r and four columns: four
      // independent sums share each X[r][m].  All outputs stay in registers until every
      // thread has finished reading T, then they overwrite it.
      float o4[2][4];
      const int items = j0 * (CNB / 4);
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int e = tid + q * 512;
#pragma unroll
        for (int u = 0; u < 4; ++u) o4[q][u] = 0.f;
        if (e < items) {
          const int r = e >> 2, c0 = j0 + ((e & 3) << 2);
          for (int mm = r; mm < j0; ++mm) {
            const float xv = A[r * ld + mm];
            const float* trow = A + mm * ld + c0;
#pragma unroll
            for (int u = 0; u < 4; ++u) o4[q][u] = fmaf(xv, trow[u], o4[q][u]);
          }
        }
      }
      __syncthreads();
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int e = tid + q * 512;
        if (e < items) {
          const int r = e >> 2, c0 = j0 + ((e & 3) << 2);
#pragma unroll
          for (int u = 0; u < 4; ++u)
            if (c0 + u < j1) A[r * ld + c0 + u] = -o4[q][u];
        }
      }
      __syncthreads();
    }
  }
  // RinvT[c][m] = X[m][c] for m <= c, zero otherwise
  float* out = RinvT + b * kk;
  for (int e = tid; e < (int)kk; e += 512) {
    const int c = e / k, mrow = e - c * k;
    out[e] = (mrow <= c) ? A[mrow * ld + c] : 0.f;
  }
}

// ==========================================================================================
// The same job for k a multiple of 16, laid out so that no step waits on a chain of dependent
// shared-memory reads and no warp reads a bank twice:
//   * the warp that factors a diagonal block R_JJ also inverts it (reciprocal square roots are
//     kept, nothing divides); D_J = R_JJ^{-1} then does the rest as products:
//   * block row     R[J, c]  = D_J^T S[J, c]                 (512 threads: column x 4 outputs)
//   * trailing      S[r, c] -= sum_i R[i, r] R[i, c]         (a warp owns 4 rows x 32-column
//     blocks on or right of the diagonal; lanes run along columns; the 4 row entries come as
//     one 16-byte read from an aligned copy P of the block row)
//   * inverse       X[0:j0, J] = -X[0:j0, 0:j0] (R[0:j0, J] D_J), the inner product unrolled by
//     four so that its reads are in flight together.
// ==========================================================================================
// KT = k when it is known at compile time (every shared-memory address then folds into an
// immediate offset, which halves the instruction count), 0 for any k.
template <int KT>
__global__ void __launch_bounds__(512) chol_inv_fast_kernel(const float* __restrict__ S,
                                                           float* __restrict__ RinvT, int k_rt,
                                                           float shift_rel,
                                                           int32_t* __restrict__ status,
                                                           int nparts) {
  const int k = KT ? KT : k_rt;
  extern __shared__ __align__(16) float fsm[];
  __shared__ float s_red[16];
  __shared__ float s_row[2][CNB];
  __shared__ int s_bad;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ld = k | 1;
  const int nblk = k / CNB;
  const int PW = k;                       // row length of P (k is a multiple of 16)
  float* P = fsm;                          // [16][PW] block row, later [<= k][16] the product T
  float* Dinv = P + CNB * PW;              // [nblk][16][16] inverses of the diagonal blocks
  float* TB = Dinv + nblk * CNB * CNB;     // [k][16] the product T = R[0:j0, J] D_J of the inverse
  float* A = TB + CNB * k;                 // [k][ld]
  const size_t kk = (size_t)k * k;
  const float* Sb = S + (size_t)b * nparts * kk;  // S arrives as nparts parts to be added up

  float md = 0.f;
  for (int i = tid; i < k; i += 512) {
    float dsum = 0.f;
    for (int q = 0; q < nparts; ++q) dsum += __ldg(Sb + q * kk + (size_t)i * k + i);
    md = fmaxf(md, dsum);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) md = fmaxf(md, __shfl_xor_sync(0xffffffffu, md, o));
  if (lane == 0) s_red[warp] = md;
  if (tid == 0) s_bad = 0;
  __syncthreads();
  md = s_red[0];
  for (int w = 1; w < 16; ++w) md = fmaxf(md, s_red[w]);
  const float shift = shift_rel * md;
  const float tiny = fmaxf(md, 1e-30f) * 1e-12f;
  {
    // parts are added in the order 0, 1, 2, 3; two trips' worth of loads are in flight together
    const float4* S4 = reinterpret_cast<const float4*>(Sb);
    const int kv = k >> 2, nv = (int)(kk >> 2);
    auto put = [&](int e, const float4& v) {
      const int r = e / kv, c = (e - r * kv) * 4;
      float* dst = A + r * ld + c;
      dst[0] = v.x + (r == c ? shift : 0.f);
      dst[1] = v.y + (r == c + 1 ? shift : 0.f);
      dst[2] = v.z + (r == c + 2 ? shift : 0.f);
      dst[3] = v.w + (r == c + 3 ? shift : 0.f);
    };
    if (nparts == 4) {
      for (int e = tid; e < nv; e += 1024) {
        const int e2 = e + 512;
        const bool two = e2 < nv;
        float4 p[4], q[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          p[i] = __ldg(S4 + (size_t)i * nv + e);
          q[i] = two ? __ldg(S4 + (size_t)i * nv + e2) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        put(e, make_float4(((p[0].x + p[1].x) + p[2].x) + p[3].x, ((p[0].y + p[1].y) + p[2].y) + p[3].y,
                           ((p[0].z + p[1].z) + p[2].z) + p[3].z, ((p[0].w + p[1].w) + p[2].w) + p[3].w));
        if (two)
          put(e2, make_float4(((q[0].x + q[1].x) + q[2].x) + q[3].x, ((q[0].y + q[1].y) + q[2].y) + q[3].y,
                              ((q[0].z + q[1].z) + q[2].z) + q[3].z, ((q[0].w + q[1].w) + q[2].w) + q[3].w));
      }
    } else {
      for (int e = tid; e < nv; e += 512) {
        float4 v = __ldg(S4 + e);
        for (int q = 1; q < nparts; ++q) {
          const float4 pp = __ldg(S4 + (size_t)q * nv + e);
          v.x += pp.x; v.y += pp.y; v.z += pp.z; v.w += pp.w;
        }
        put(e, v);
      }
    }
  }
  __syncthreads();

  // ---------------- phase 1: Cholesky, R^T R = S + shift I ----------------
  // One warp factors and inverts a diagonal block; so that the others need not wait for it, the
  // trailing update of a block column first brings the rows of the next diagonal block up to
  // date, and that block is then factored while the rest of the update runs.
  auto diag = [&](int jb) {
    const int j0 = jb * CNB;
    float* Dj = Dinv + jb * CNB * CNB;
    // lane c (< 16) keeps column c of the diagonal block
    float col[CNB], rd[CNB];
    const int gc = j0 + (lane & 15);
#pragma unroll
    for (int r = 0; r < CNB; ++r) col[r] = (r <= (lane & 15)) ? A[(j0 + r) * ld + gc] : 0.f;
#pragma unroll
    for (int i = 0; i < CNB; ++i) {
      float piv = __shfl_sync(0xffffffffu, col[i], i);
      if (!(piv > 0.f)) {
        piv = tiny;
        if (lane == 0) s_bad = 1;
      }
      const float rinv = rsqrtf(piv);
      rd[i] = rinv;  // 1 / R_ii, the same in every lane
      if ((lane & 15) == i) col[i] = piv * rinv;
      else if ((lane & 15) > i) col[i] = col[i] * rinv;
      if (lane < CNB) s_row[i & 1][lane] = col[i];
      __syncwarp();
#pragma unroll
      for (int r = i + 1; r < CNB; ++r) {
        const float v = s_row[i & 1][r];
        if ((lane & 15) >= r) col[r] = fmaf(-v, col[i], col[r]);
      }
    }
    if (lane < CNB) {
#pragma unroll
      for (int r = 0; r < CNB; ++r)
        if (r <= lane) A[(j0 + r) * ld + gc] = col[r];
    }
    __syncwarp();
    // lane c solves R_JJ x = e_c by back substitution: x_c = 1/R_cc,
    // x_i = -(1/R_ii) sum_{i < mm <= c} R[i][mm] x_mm.  Row entries are broadcast reads.
    float x[CNB];
#pragma unroll
    for (int i = 0; i < CNB; ++i) x[i] = 0.f;
    const int c = lane & 15;
#pragma unroll
    for (int i = CNB - 1; i >= 0; --i) {
      float sacc = 0.f;
#pragma unroll
      for (int mm = i + 1; mm < CNB; ++mm) sacc = fmaf(A[(j0 + i) * ld + j0 + mm], x[mm], sacc);
      x[i] = (i == c) ? rd[i] : ((i < c) ? -rd[i] * sacc : 0.f);
    }
    if (lane < CNB) {
#pragma unroll
      for (int i = 0; i < CNB; ++i) Dj[i * CNB + c] = x[i];
    }
  };
  // one 4-row x 32-column unit of the trailing update of block column jb (P = its block row)
  auto trail_unit = [&](int j1, int m, int r0, int u) {
    const int cl = u * 32 + lane;
    const bool on = cl < m;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < CNB; ++i) {
      const float4 a4 = *reinterpret_cast<const float4*>(P + i * PW + r0);
      const float bv = on ? P[i * PW + cl] : 0.f;
      acc[0] = fmaf(a4.x, bv, acc[0]);
      acc[1] = fmaf(a4.y, bv, acc[1]);
      acc[2] = fmaf(a4.z, bv, acc[2]);
      acc[3] = fmaf(a4.w, bv, acc[3]);
    }
#pragma unroll
    for (int xx = 0; xx < 4; ++xx)
      if (on && r0 + xx < m && cl >= r0 + xx) A[(j1 + r0 + xx) * ld + j1 + cl] -= acc[xx];
  };
  // ---- the inverse X = R^{-1}, in place, one block column J per step of the factorisation:
  //        X[0:j0, J] = -X[0:j0, 0:j0] (R[0:j0, J] D_J),   X_JJ = D_J.
  //      Step J reads rows of R above block row J (final since step J - 1), D_J (from the
  //      look-ahead of step J - 1) and the block columns of X before J, and writes only above
  //      block row J, where the factorisation no longer looks: it runs inside step J of the
  //      factorisation, on the warps that the shrinking trailing update leaves idle.
  // T = R[0:j0, J] D_J, all threads
  auto inv_T = [&](int j0, const float* Dj) {
    for (int rb = 0; rb < j0; rb += 128) {
      const int r = rb + (tid >> 2), cg = tid & 3;
      if (r < j0) {
        float out[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int mm = 0; mm < CNB; ++mm) {
          const float rv = A[r * ld + j0 + mm];
          const float4 d4 = *reinterpret_cast<const float4*>(Dj + mm * CNB + 4 * cg);
          out[0] = fmaf(rv, d4.x, out[0]);
          out[1] = fmaf(rv, d4.y, out[1]);
          out[2] = fmaf(rv, d4.z, out[2]);
          out[3] = fmaf(rv, d4.w, out[3]);
        }
        *reinterpret_cast<float4*>(TB + r * CNB + 4 * cg) = make_float4(out[0], out[1], out[2], out[3]);
      }
    }
  };
  // X[r][J] = - sum_{mm = r}^{j0 - 1} X[r][mm] T[mm][:] and X_JJ = D_J, warps 1 .. 15
  auto inv_X = [&](int j0, const float* Dj) {
    const int t2 = tid - 32;  // 0 .. 479
    for (int rb = 0; rb < j0; rb += 120) {
      const int r = rb + (t2 >> 2), cg = t2 & 3;
      if (r < j0) {
        float o0[4] = {0.f, 0.f, 0.f, 0.f}, o1[4] = {0.f, 0.f, 0.f, 0.f};
        const float* xr = A + r * ld;
        const float* tb = TB + 4 * cg;
        // the eight rows of a warp walk the same mm (from the first of them on, entries left
        // of a row's diagonal counting as zero), so that lanes with the same columns read the
        // same 16 bytes of T
        int mm = r & ~7;
        for (; mm + 3 < j0; mm += 4) {
          const float x0 = (mm >= r) ? xr[mm] : 0.f, x1 = (mm + 1 >= r) ? xr[mm + 1] : 0.f;
          const float x2 = (mm + 2 >= r) ? xr[mm + 2] : 0.f, x3 = (mm + 3 >= r) ? xr[mm + 3] : 0.f;
          const float4 t0 = *reinterpret_cast<const float4*>(tb + mm * CNB);
          const float4 t1 = *reinterpret_cast<const float4*>(tb + (mm + 1) * CNB);
          const float4 t2v = *reinterpret_cast<const float4*>(tb + (mm + 2) * CNB);
          const float4 t3 = *reinterpret_cast<const float4*>(tb + (mm + 3) * CNB);
          o0[0] = fmaf(x0, t0.x, o0[0]); o0[1] = fmaf(x0, t0.y, o0[1]);
          o0[2] = fmaf(x0, t0.z, o0[2]); o0[3] = fmaf(x0, t0.w, o0[3]);
          o1[0] = fmaf(x1, t1.x, o1[0]); o1[1] = fmaf(x1, t1.y, o1[1]);
          o1[2] = fmaf(x1, t1.z, o1[2]); o1[3] = fmaf(x1, t1.w, o1[3]);
          o0[0] = fmaf(x2, t2v.x, o0[0]); o0[1] = fmaf(x2, t2v.y, o0[1]);
          o0[2] = fmaf(x2, t2v.z, o0[2]); o0[3] = fmaf(x2, t2v.w, o0[3]);
          o1[0] = fmaf(x3, t3.x, o1[0]); o1[1] = fmaf(x3, t3.y, o1[1]);
          o1[2] = fmaf(x3, t3.z, o1[2]); o1[3] = fmaf(x3, t3.w, o1[3]);
        }
        for (; mm < j0; ++mm) {
          const float x0 = (mm >= r) ? xr[mm] : 0.f;
          const float4 t0 = *reinterpret_cast<const float4*>(tb + mm * CNB);
          o0[0] = fmaf(x0, t0.x, o0[0]); o0[1] = fmaf(x0, t0.y, o0[1]);
          o0[2] = fmaf(x0, t0.z, o0[2]); o0[3] = fmaf(x0, t0.w, o0[3]);
        }
        // columns J of these rows are read by nobody in this part of the step
#pragma unroll
        for (int u = 0; u < 4; ++u) A[r * ld + j0 + 4 * cg + u] = -(o0[u] + o1[u]);
      }
    }
    if (t2 < CNB * CNB) {
      const int i = t2 >> 4, c = t2 & 15;
      A[(j0 + i) * ld + j0 + c] = Dj[i * CNB + c];
    }
  };
  if (warp == 0) diag(0);
  __syncthreads();
  for (int jb = 0; jb < nblk; ++jb) {
    const int j0 = jb * CNB, j1 = j0 + CNB, m = k - j1;
    float* Dj = Dinv + jb * CNB * CNB;
    // block row: R[j0 + i][c] = sum_{mm <= i} D[mm][i] S[j0 + mm][c] for c >= j1.
    // thread = (column, group ig of four outputs i = 4 ig ..); 128 columns per pass.
    for (int cb = 0; cb < m; cb += 128) {
      const int cl = cb + (tid & 127), ig = tid >> 7;
      const bool on = cl < m;
      float a[CNB], out[4] = {0.f, 0.f, 0.f, 0.f};
      if (on) {
#pragma unroll
        for (int mm = 0; mm < CNB; ++mm)
          a[mm] = (mm <= 4 * ig + 3) ? A[(j0 + mm) * ld + j1 + cl] : 0.f;
#pragma unroll
        for (int mm = 0; mm < CNB; ++mm) {
          if (mm <= 4 * ig + 3) {
            const float4 d4 = *reinterpret_cast<const float4*>(Dj + mm * CNB + 4 * ig);
            out[0] = fmaf(d4.x, a[mm], out[0]);
            out[1] = fmaf(d4.y, a[mm], out[1]);
            out[2] = fmaf(d4.z, a[mm], out[2]);
            out[3] = fmaf(d4.w, a[mm], out[3]);
          }
        }
      }
      __syncthreads();  // every input of this pass has been read
      if (on) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          A[(j0 + 4 * ig + u) * ld + j1 + cl] = out[u];
          P[(4 * ig + u) * PW + cl] = out[u];
        }
      }
    }
    __syncthreads();
    // trailing update, first the rows of the next diagonal block (four strips of four rows)
    {
      const int nu = (m + 31) >> 5;
      const int n_first = min(4, m >> 2) * nu;
      for (int id = warp; id < n_first; id += 16) {
        const int s4 = id / nu, u = id - s4 * nu;
        if (u >= ((4 * s4) >> 5)) trail_unit(j1, m, 4 * s4, u);
      }
    }
    inv_T(j0, Dj);
    __syncthreads();
    if (warp == 0) {
      if (jb + 1 < nblk) diag(jb + 1);
    } else {
      for (int s4 = 4 + (warp - 1); s4 * 4 < m; s4 += 15)
        for (int u = (4 * s4) >> 5; u * 32 < m; ++u) trail_unit(j1, m, 4 * s4, u);
      inv_X(j0, Dj);
    }
    __syncthreads();
  }
  if (tid == 0 && s_bad) atomicMax(&status[b], (int)TC_ERR_BREAKDOWN);

  // RinvT[c][m] = X[m][c] for m <= c, zero otherwise
  float* out = RinvT + b * kk;
  for (int e = tid; e < (int)kk; e += 512) {
    const int c = e / k, mrow = e - c * k;
    out[e] = (mrow <= c) ? A[mrow * ld + c] : 0.f;
  }
}

// ==========================================================================================
// One-sided Jacobi eigen-solver for a symmetric positive semi-definite n x n matrix.
// One block (16 warps) per image.  W (column-major) starts as the matrix, J as the identity;
// each pair step rotates columns p, q of both so that the W columns become orthogonal.  At
// convergence  W = Z Theta  and  J = Z  (eigenvectors), column norms = eigenvalues.
// Pairs follow a round-robin tournament: n/2 disjoint pairs per round, one warp per pair,
// a block barrier between rounds.  R = elements of a column each lane keeps in registers.
// ==========================================================================================
template <int R>
__device__ inline int jacobi_pair(float* __restrict__ W, float* __restrict__ J, int n, int p,
                                  int q, int lane, float tol, float floor2,
                                  float count_floor2) {
  float wp[R], wq[R];
  float a = 0.f, bq = 0.f, g = 0.f;
  float* Wp = W + (size_t)p * n;
  float* Wq = W + (size_t)q * n;
#pragma unroll
  for (int i = 0; i < R; ++i) {
    const int r = lane + 32 * i;
    wp[i] = (r < n) ? Wp[r] : 0.f;
    wq[i] = (r < n) ? Wq[r] : 0.f;
    a = fmaf(wp[i], wp[i], a);
    bq = fmaf(wq[i], wq[i], bq);
    g = fmaf(wp[i], wq[i], g);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    a += __shfl_xor_sync(0xffffffffu, a, o);
    bq += __shfl_xor_sync(0xffffffffu, bq, o);
    g += __shfl_xor_sync(0xffffffffu, g, o);
  }
  const float nn = sqrtf(a) * sqrtf(bq);
  if (!(fabsf(g) > tol * nn) || !(fmaxf(a, bq) > floor2)) return 0;
  const float zeta = (bq - a) / (2.0f * g);
  const float t = copysignf(1.0f, zeta) / (fabsf(zeta) + sqrtf(fmaf(zeta, zeta, 1.0f)));
  const float c = rsqrtf(fmaf(t, t, 1.0f));
  const float s = c * t;
#pragma unroll
  for (int i = 0; i < R; ++i) {
    const int r = lane + 32 * i;
    if (r < n) {
      Wp[r] = c * wp[i] - s * wq[i];
      Wq[r] = fmaf(s, wp[i], c * wq[i]);
    }
  }
  float* Jp = J + (size_t)p * n;
  float* Jq = J + (size_t)q * n;
#pragma unroll
  for (int i = 0; i < R; ++i) {
    const int r = lane + 32 * i;
    if (r < n) {
      const float jp = Jp[r], jq = Jq[r];
      Jp[r] = c * jp - s * jq;
      Jq[r] = fmaf(s, jp, c * jq);
    }
  }
  // a rotation between two columns that both lie under the rank cut-off does not delay
  // convergence: neither column enters Eq. 3-6
  return fmaxf(a, bq) > count_floor2 ? 1 : 0;
}

template <int R>
__global__ void __launch_bounds__(512) jacobi_kernel(const float* __restrict__ Hin,
                                                    float* __restrict__ Wg, float* __restrict__ ZTg,
                                                    float* __restrict__ theta, int n,
                                                    int max_sweeps, float tol, int use_smem,
                                                    int32_t* __restrict__ status, float floor_rel,
                                                    float count_rel) {
  extern __shared__ float sm[];
  __shared__ int s_rot;
  __shared__ float s_red[16];
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t nn = (size_t)n * n;
  const float* Hb = Hin + b * nn;
  float* W = use_smem ? sm : Wg + b * nn;
  float* J = use_smem ? sm + nn : ZTg + b * nn;

  // W = (H + H^T) / 2 (column-major == row-major for a symmetric matrix), J = I
  float md = 0.f;
  for (size_t e = tid; e < nn; e += 512) {
    const int p = (int)(e / n), i = (int)(e % n);
    const float v = 0.5f * (Hb[e] + Hb[(size_t)i * n + p]);
    W[e] = v;
    J[e] = (p == i) ? 1.f : 0.f;
    if (p == i) md = fmaxf(md, fabsf(v));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) md = fmaxf(md, __shfl_xor_sync(0xffffffffu, md, o));
  if (lane == 0) s_red[warp] = md;
  if (tid == 0) s_rot = 0;
  __syncthreads();
  md = s_red[0];
  for (int w = 1; w < 16; ++w) md = fmaxf(md, s_red[w]);
  // column pairs whose norms (eigenvalue estimates) are BOTH below the floor are left alone:
  // they are rounding noise of the largest eigenvalue, or lie below the rank cut-off, and
  // rotating them against each other only slows convergence
  const float floor1 = floor_rel * md;
  const float floor2 = floor1 * floor1;
  const float count_floor2 = (count_rel * md) * (count_rel * md);

  const int ne = (n + 1) & ~1;  // even number of players; index n (if any) is a bye
  const int m = ne - 1;
  const int half = ne / 2;
  int sweep = 0;
  bool converged = false;
  for (; sweep < max_sweeps; ++sweep) {
    int rot = 0;
    for (int round = 0; round < m; ++round) {
      for (int slot = warp; slot < half; slot += 16) {
        int u, v;
        if (slot == 0) {
          u = round;
          v = m;
        } else {
          u = round + slot;
          if (u >= m) u -= m;
          v = round - slot;
          if (v < 0) v += m;
        }
        if (u >= n || v >= n) continue;
        const int p = min(u, v), q = max(u, v);
        rot += jacobi_pair<R>(W, J, n, p, q, lane, tol, floor2, count_floor2);
      }
      __syncthreads();
    }
    if (lane == 0 && rot) atomicAdd(&s_rot, rot);
    __syncthreads();
    const int total = s_rot;
    __syncthreads();
    if (tid == 0) s_rot = 0;
    if (total == 0) {
      converged = true;
      break;
    }
  }
  __syncthreads();
  if (tid == 0 && !converged) atomicMax(&status[b], (int)TC_ERR_NOT_CONVERGED);

  // eigenvalues = column norms of W;  eigenvectors = columns of J, written as ZT[p][i]
  for (int p = warp; p < n; p += 16) {
    float a = 0.f;
    for (int r = lane; r < n; r += 32) {
      const float v = W[(size_t)p * n + r];
      a = fmaf(v, v, a);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if (lane == 0) theta[(size_t)b * n + p] = sqrtf(a);
  }
  if (use_smem) {
    float* out = ZTg + b * nn;
    for (size_t e = tid; e < nn; e += 512) out[e] = J[e];
  }
}

// ==========================================================================================
// Symmetric eigen-solver for matrices that fit in shared memory (n <= ~230):
//   1. Householder reduction to a tridiagonal matrix T, the orthogonal factor Q formed in place;
//   2. every eigenvalue of T by bisection on the Sturm count, one thread per eigenvalue;
//   3. the eigenvector of T for every eigenvalue that can pass the rank cut-off, by inverse
//      iteration (tridiagonal elimination with partial pivoting), one thread per eigenvalue,
//      its four work vectors in global scratch laid out thread-fastest;
//   4. eigenvalues refined as Rayleigh quotients on T, eigenvectors of H as Z = Q Y.
// Nothing here is a serial recurrence over the whole matrix, which is what makes it several
// times faster than sweeping Jacobi rotations or chasing QL bulges from one thread.
// Eigenvectors of eigenvalues closer together than the rounding level of T are not
// re-orthogonalised against each other (Eq. 3-6 is not unique there in the first place).
//   in   H [n][n] symmetric (only its symmetric part is used)
//   out  theta [n] eigenvalues (ascending), ZT [n][n] with ZT[p][i] = component i of
//        eigenvector p (all zero for eigenvalues under a quarter of the rank cut-off)
//   scratch u0, u1, u2, yv, ml: [n][n] float each, per image
// One block (16 warps) per image.
// ==========================================================================================
// Barrier among `count` threads (a multiple of 32) of the block, on hardware barrier `id` (1..15).
__device__ __forceinline__ void bar_named(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

template <int NT>  // n when it is known at compile time (addresses fold into immediates), else 0
__global__ void __launch_bounds__(512) tridiag_eig_kernel(const float* Hin,
                                                         float* __restrict__ ZTg,
                                                         float* __restrict__ theta, int n_rt, float rank_tol,
                                                         float* __restrict__ u0g, float* __restrict__ u1g,
                                                         float* __restrict__ u2g, float* yg, float* __restrict__ mlg,
                                                         size_t ml_stride,
                                                         int32_t* __restrict__ status, int nparts,
                                                         int emit_factors) {
  // emit_factors: instead of Z = Q Y the kernel leaves its two factors for the tensor-core
  // products: ZTg receives Q^T ([j][i] = Q[i][j]) and u0g receives Y^T ([p][j] = component j of
  // the eigenvector p of T)
  const int n = NT ? NT : n_rt;
  extern __shared__ __align__(16) float sm[];
  const int ld = n | 1;
  const int n4 = (n + 3) & ~3;         // the vectors start on 16-byte boundaries
  float* dv = sm;                      // [n] diagonal
  float* ev = dv + n4;                 // [n] sub-diagonal (ev[i] couples i and i+1)
  float* vv = ev + n4;                 // [n] Householder vector of the current step
  float* vv2 = vv + n4;                // [n] ... of the next step (the two alternate)
  float* pv = vv2 + n4;                // [n] work vector
  float* beta = pv + n4;               // [n] reflector scales
  float* dn = beta + n4;               // [n] diagonal of T / |T| for the Sturm counts
  float2* cs = reinterpret_cast<float2*>(dn + n4);     // [4 n floats] partial sums of the reduction
  float* qf = reinterpret_cast<float*>(cs) + 4 * n4;   // [16 n] reflector block and partial products
  float* A = qf + 16 * n4;             // [n][ld]
  __shared__ float s_red[16];
  __shared__ int s_fail;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* Hb = Hin + (size_t)b * nparts * n * n;  // H arrives as nparts parts to be added up

  if (nparts == 4 && (n & 3) == 0) {
    // the parts come from the kernel that writes every entry and its mirror image with the
    // same bits, so their sum is symmetric as it stands
    const float4* H4 = reinterpret_cast<const float4*>(Hb);
    const int kv = n >> 2, nv = (n * n) >> 2;
    for (int e = tid; e < nv; e += 1024) {  // two trips' worth of loads in flight together
      const int e2 = e + 512;
      const bool two = e2 < nv;
      float4 p[4], q[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        p[i] = __ldg(H4 + (size_t)i * nv + e);
        q[i] = two ? __ldg(H4 + (size_t)i * nv + e2) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
      {
        const int r = e / kv, c = (e - r * kv) * 4;
        float* dst = A + r * ld + c;
        dst[0] = (p[0].x + p[1].x) + (p[2].x + p[3].x);
        dst[1] = (p[0].y + p[1].y) + (p[2].y + p[3].y);
        dst[2] = (p[0].z + p[1].z) + (p[2].z + p[3].z);
        dst[3] = (p[0].w + p[1].w) + (p[2].w + p[3].w);
      }
      if (two) {
        const int r = e2 / kv, c = (e2 - r * kv) * 4;
        float* dst = A + r * ld + c;
        dst[0] = (q[0].x + q[1].x) + (q[2].x + q[3].x);
        dst[1] = (q[0].y + q[1].y) + (q[2].y + q[3].y);
        dst[2] = (q[0].z + q[1].z) + (q[2].z + q[3].z);
        dst[3] = (q[0].w + q[1].w) + (q[2].w + q[3].w);
      }
    }
  } else if (nparts == 1 && (n & 3) == 0) {
    // one part that need not be symmetric to the last bit (a product Q^T (G Q)): 16-byte loads,
    // then the two triangles are averaged in shared memory
    const float4* H4 = reinterpret_cast<const float4*>(Hb);
    const int kv = n >> 2, nv = (n * n) >> 2;
    for (int e = tid; e < nv; e += 512) {
      const float4 p = __ldg(H4 + e);
      const int r = e / kv, c = (e - r * kv) * 4;
      float* dst = A + r * ld + c;
      dst[0] = p.x; dst[1] = p.y; dst[2] = p.z; dst[3] = p.w;
    }
    __syncthreads();
    for (int e = tid; e < n * n; e += 512) {
      const int r = e / n, c = e - r * n;
      if (c > r) {
        const float m = 0.5f * (A[r * ld + c] + A[c * ld + r]);
        A[r * ld + c] = m;
        A[c * ld + r] = m;
      }
    }
  } else {
    for (int e = tid; e < n * n; e += 512) {
      const int r = e / n, c = e - r * n;
      float h = 0.f, ht = 0.f;
      for (int q = 0; q < nparts; ++q) {
        h += Hb[(size_t)q * n * n + e];
        ht += Hb[(size_t)q * n * n + (size_t)c * n + r];
      }
      A[r * ld + c] = 0.5f * (h + ht);
    }
  }
  if (tid == 0) s_fail = 0;
  __syncthreads();

  // ---------------- Householder tridiagonalisation ----------------
  // Three block barriers per column and no warp reductions inside the O(m^2) parts: a thread
  // owns one column c of the trailing block and a range of its rows (the block is symmetric, so
  // the column sum over that range is a partial of (B v)_c); the ranges are combined through
  // shared memory.  While the trailing block is updated, the thread that owns its first column
  // also writes that column out as the next step's vector and gathers its |x|^2, so a step
  // starts with everything it needs except the square root, which every thread takes itself.
  // Vector entries are read four at a time (one broadcast load per four rows).
  // The scalar parts of a step are repeated by every warp, four warps to a scheduler, so what
  // counts there is the number of instructions: sums come as one or two 16-byte loads, the
  // square root and the reciprocal as a Newton step on the hardware approximations.
  __shared__ float s_sig[16];
  __shared__ __align__(16) float s_sig4[4];  // |x|^2 of the next column, one partial per row range
  __shared__ __align__(16) float s_red8[8];  // v.p, one partial per warp of the first row range
  float* part = reinterpret_cast<float*>(cs);  // [<= 4][n] partial products (cs is free here)
  if (warp == 0) {
    float ps = 0.f;
    for (int r = lane; r + 1 < n; r += 32) {
      const float x = A[(1 + r) * ld];
      vv[r] = x;
      ps = fmaf(x, x, ps);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
    if (lane < 4) s_sig4[lane] = (lane == 0) ? ps : 0.f;
  }
  __syncthreads();
  int cw = 0, G = 1, g = 0, c = 0;  // thread layout: cw warps cover the columns, G row ranges
  bool lead = false;                // this warp holds column 0 of its row range
  for (int j = 0; j + 2 < n; ++j) {
    const int m = n - j - 1;  // order of the trailing block B = A[j+1.., j+1..]
    float* vc = (j & 1) ? vv2 : vv;  // x of this step (v is x with v_0 in place of its entry 0)
    float* vn = (j & 1) ? vv : vv2;  // x of the next step
    const float4 s4 = *reinterpret_cast<const float4*>(s_sig4);
    const float sigma = (s4.x + s4.y) + (s4.z + s4.w);
    const float x0 = vc[0];
    const float tail = sigma - x0 * x0;  // |x|^2 without its first entry
    // reflector H = I - bj v v^T with v = x - alpha e_1; a column already in tridiagonal form
    // gets bj = 0 (H = I) and keeps its entries
    const bool skip = !(tail > 1e-30f * sigma) || !(sigma > 0.f);
    const float rs = rsqrtf(sigma);
    float nrm = sigma * rs;
    nrm = fmaf(fmaf(-nrm, nrm, sigma), 0.5f * rs, nrm);
    const float alpha = skip ? x0 : -copysignf(nrm, x0);
    const float v0 = skip ? x0 : x0 - alpha;
    const float den = tail + v0 * v0;
    float rc = __fdividef(2.0f, den);
    rc = fmaf(fmaf(-den, rc, 2.0f), 0.5f * rc, rc);
    const float bj = skip ? 0.f : rc;
    if (tid == 0) {
      dv[j] = A[j * ld + j];
      ev[j] = alpha;
      beta[j] = bj;
    }
    if (((m + 31) >> 5) != cw) {
      cw = (m + 31) >> 5;
      G = min(4, 16 / cw);
      g = warp / cw;
      c = (warp - g * cw) * 32 + lane;
      lead = (warp == g * cw);
    }
    const bool on = (g < G) && (c < m);
    // rows per range, a multiple of four (G is 2, 3 or 4; the multiplication is a division by 3)
    const int per0 = (G == 4) ? (m + 3) >> 2 : (G == 3) ? ((m + 2) * 21846) >> 16 : (m + 1) >> 1;
    const int per = (per0 + 3) & ~3;
    const int r_lo = g * per, r_hi = min(m, r_lo + per);
    float* colp = A + (j + 1) * ld + j + 1 + c;  // B[0][c]; rows are ld apart
    if (on) {
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
      int r = r_lo;
      const float* bp = colp + r_lo * ld;
      for (; r + 3 < r_hi; r += 4, bp += 4 * ld) {
        float4 v4 = *reinterpret_cast<const float4*>(vc + r);
        if (r == 0) v4.x = v0;
        a0 = fmaf(bp[0], v4.x, a0);
        a1 = fmaf(bp[ld], v4.y, a1);
        a2 = fmaf(bp[2 * ld], v4.z, a2);
        a3 = fmaf(bp[3 * ld], v4.w, a3);
      }
      for (; r < r_hi; ++r) a0 = fmaf(colp[r * ld], (r == 0) ? v0 : vc[r], a0);
      part[g * n + c] = (a0 + a1) + (a2 + a3);
    }
    __syncthreads();
    // p = bj * B v ; v.p
    float vpp = 0.f;
    if (g == 0 && c < m) {
      const float t0 = part[c], t1 = part[n + c];
      const float t2 = (G > 2) ? part[2 * n + c] : 0.f, t3 = (G > 3) ? part[3 * n + c] : 0.f;
      const float pc = bj * ((t0 + t1) + (t2 + t3));
      pv[c] = pc;
      vpp = ((c == 0) ? v0 : vc[c]) * pc;
    }
    // the column is kept for the accumulation of Q (everyone has read its x_0 by now)
    if (tid == 0) A[(j + 1) * ld + j] = v0;
    if (warp < 8) {  // the first row range is at most seven warps; the others hold zero
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) vpp += __shfl_xor_sync(0xffffffffu, vpp, o);
      if (lane == 0) s_red8[warp] = vpp;
    }
    __syncthreads();
    const float4 ra = *reinterpret_cast<const float4*>(s_red8);
    const float4 rb = *reinterpret_cast<const float4*>(s_red8 + 4);
    const float vp = ((ra.x + ra.y) + (ra.z + ra.w)) + ((rb.x + rb.y) + (rb.z + rb.w));
    const float K = 0.5f * bj * vp;  // w = p - K v
    // B -= v w^T + w v^T ; column 0 of the new B, below its top entry, is the next x
    float sig_part = 0.f;
    auto update = [&](auto tag) {
      constexpr bool LEAD = decltype(tag)::value;  // this warp's lane 0 owns column 0
      const bool first = LEAD && (lane == 0);
      const float vcc = (c == 0) ? v0 : vc[c], wc = fmaf(-K, vcc, pv[c]);
      int r = r_lo;
      float* bp = colp + r_lo * ld;
      for (; r + 3 < r_hi; r += 4, bp += 4 * ld) {
        float4 v4 = *reinterpret_cast<const float4*>(vc + r);
        if (r == 0) v4.x = v0;
        const float4 p4 = *reinterpret_cast<const float4*>(pv + r);
        const float vr[4] = {v4.x, v4.y, v4.z, v4.w};
        const float pr[4] = {p4.x, p4.y, p4.z, p4.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float wr = fmaf(-K, vr[u], pr[u]);
          const float nv = bp[u * ld] - fmaf(vr[u], wc, wr * vcc);
          bp[u * ld] = nv;
          if (LEAD) {
            if (first && r + u >= 1) {
              vn[r + u - 1] = nv;
              sig_part = fmaf(nv, nv, sig_part);
            }
          }
        }
      }
      for (; r < r_hi; ++r) {
        const float vr = (r == 0) ? v0 : vc[r], wr = fmaf(-K, vr, pv[r]);
        const float nv = colp[r * ld] - fmaf(vr, wc, wr * vcc);
        colp[r * ld] = nv;
        if (LEAD) {
          if (first && r >= 1) {
            vn[r - 1] = nv;
            sig_part = fmaf(nv, nv, sig_part);
          }
        }
      }
    };
    if (on) {
      if (lead) update(std::true_type{}); else update(std::false_type{});
    }
    if (lead && lane == 0 && g < 4) s_sig4[g] = sig_part;  // zero from a range that is not in use
    __syncthreads();
  }
  if (tid == 0) {
    if (n >= 2) {
      dv[n - 2] = A[(n - 2) * ld + n - 2];
      ev[n - 2] = A[(n - 1) * ld + n - 2];
      beta[n - 2] = 0.f;
    }
    dv[n - 1] = A[(n - 1) * ld + n - 1];
    ev[n - 1] = 0.f;
    A[(n - 1) * ld + n - 1] = 1.f;  // the accumulation of Q starts from the identity
  }
  __syncthreads();

  // From here the block works as two teams until Z = Q Y needs both results: the first
  // ceil(n / 32) warps find the eigenpairs of T (one thread per eigenvalue; they only read the
  // diagonals of T), the other warps accumulate Q.  Each team synchronises on its own barrier.
  const int nbw = (n + 31) >> 5;           // warps of the eigenvalue team
  const int ET = nbw * 32;                 // its threads
  const int NQW = 16 - nbw, QT = NQW * 32; // warps and threads of the Q team
  const int qt = tid - ET, qw = warp - nbw;
  if (warp >= nbw) {
  // ---------------- Q = H_0 H_1 ... H_{n-3}, accumulated backwards, in place ----------------
  // Reflector j sits in A[j+1.., j].  Reflectors are applied four at a time in the compact WY
  // form  H_{j0} ... H_{j1} = I - V T V^T  (T upper triangular), so a block costs three barriers
  // and two passes over the rows instead of two barriers and two passes per reflector.
  // Before a block, columns c >= j1+2 of A (rows >= j1+2) hold the product of the later
  // reflectors; everything else of Q is still the identity, which the block first writes out.
  {
    constexpr int NBQ = 4;
    float* Vb = qf;              // [n][NBQ]  Vb[r][i] = entry r of reflector j0+i (0 above its support
                                 // and for a reflector the block does not have): one 16-byte read per row
    float* Wp = qf + NBQ * n;    // [3][NBQ][n] partial products V^T Q per row range
    __shared__ float s_vv[NBQ][NBQ];  // v_a . v_b for a < b
    for (int j1 = n - 3; j1 >= 0; j1 -= NBQ) {
      const int j0 = max(0, j1 - NBQ + 1), nbk = j1 - j0 + 1;
      // (1) copy the block's reflectors out of the columns that are about to be overwritten
      for (int idx = qt; idx < NBQ * n; idx += QT) {
        const int r = idx / NBQ, i = idx - r * NBQ, jj = j0 + i;
        Vb[idx] = (i < nbk && r >= jj + 1) ? A[r * ld + jj] : 0.f;
      }
      bar_named(1, QT);
      // (2) identity columns j0+1 .. j1+1, zero rows j0+1 .. j1+1 right of them; v_a . v_b
      for (int idx = qt; idx < (n - j0 - 1) * nbk; idx += QT) {
        const int r = j0 + 1 + idx / nbk, c = j0 + 1 + idx % nbk;
        A[r * ld + c] = (r == c) ? 1.f : 0.f;
      }
      for (int idx = qt; idx < nbk * (n - j1 - 2); idx += QT) {
        const int r = j0 + 1 + idx / (n - j1 - 2), c = j1 + 2 + idx % (n - j1 - 2);
        A[r * ld + c] = 0.f;
      }
      if (qw < 6) {
        // the six pairs a < b of a block of four, one warp each
        const int a2 = (qw < 3) ? 0 : (qw < 5 ? 1 : 2);
        const int b2 = (qw < 3) ? qw + 1 : (qw < 5 ? qw - 1 : 3);
        if (b2 < nbk) {
          float d2 = 0.f;
          for (int r = lane; r < n; r += 32) d2 = fmaf(Vb[r * NBQ + a2], Vb[r * NBQ + b2], d2);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) d2 += __shfl_xor_sync(0xffffffffu, d2, o);
          if (lane == 0) s_vv[a2][b2] = d2;
        }
      }
      bar_named(1, QT);
      // (3) W = V^T Q on the columns c >= j0+1, rows split into up to three ranges
      const int ncols = n - j0 - 1;
      const int cw = (ncols + 31) >> 5;
      const int G = min(3, NQW / cw);
      const int g = qw / cw, c = j0 + 1 + (qw - g * cw) * 32 + lane;
      const bool on = (g < G) && (c < n);
      const int per = (ncols + G - 1) / G;
      const int r_lo = j0 + 1 + g * per, r_hi = min(n, r_lo + per);
      if (on) {
        float acc[NBQ] = {0.f, 0.f, 0.f, 0.f};
        for (int r = r_lo; r < r_hi; ++r) {
          const float qv = A[r * ld + c];
          const float4 v4 = *reinterpret_cast<const float4*>(Vb + r * NBQ);
          acc[0] = fmaf(v4.x, qv, acc[0]);
          acc[1] = fmaf(v4.y, qv, acc[1]);
          acc[2] = fmaf(v4.z, qv, acc[2]);
          acc[3] = fmaf(v4.w, qv, acc[3]);
        }
#pragma unroll
        for (int i = 0; i < NBQ; ++i) Wp[(g * NBQ + i) * n + c] = acc[i];
      }
      bar_named(1, QT);
      // (4) T W, (5) Q -= V (T W)
      if (on) {
        float w[NBQ], tw[NBQ];
#pragma unroll
        for (int i = 0; i < NBQ; ++i) {
          float t = 0.f;
          for (int q = 0; q < G; ++q) t += Wp[(q * NBQ + i) * n + c];
          w[i] = (i < nbk) ? t : 0.f;
        }
        // T (upper triangular, 4 x 4) of the compact WY form, in registers of every thread:
        //   T_ii = beta_i ;  T[0:i, i] = -beta_i T[0:i, 0:i] (V[:, 0:i]^T v_i)
        // (a reflector the block does not have gets beta = 0, which zeroes its row and column)
        const float b0 = beta[j0], b1 = (nbk > 1) ? beta[j0 + 1] : 0.f;
        const float b2 = (nbk > 2) ? beta[j0 + 2] : 0.f, b3 = (nbk > 3) ? beta[j0 + 3] : 0.f;
        const float v01 = (nbk > 1) ? s_vv[0][1] : 0.f;
        const float v02 = (nbk > 2) ? s_vv[0][2] : 0.f, v12 = (nbk > 2) ? s_vv[1][2] : 0.f;
        const float v03 = (nbk > 3) ? s_vv[0][3] : 0.f, v13 = (nbk > 3) ? s_vv[1][3] : 0.f;
        const float v23 = (nbk > 3) ? s_vv[2][3] : 0.f;
        const float t01 = -b1 * (b0 * v01);
        const float t02 = -b2 * fmaf(t01, v12, b0 * v02);
        const float t12 = -b2 * (b1 * v12);
        const float t03 = -b3 * fmaf(t02, v23, fmaf(t01, v13, b0 * v03));
        const float t13 = -b3 * fmaf(t12, v23, b1 * v13);
        const float t23 = -b3 * (b2 * v23);
        tw[0] = fmaf(t03, w[3], fmaf(t02, w[2], fmaf(t01, w[1], b0 * w[0])));
        tw[1] = fmaf(t13, w[3], fmaf(t12, w[2], b1 * w[1]));
        tw[2] = fmaf(t23, w[3], b2 * w[2]);
        tw[3] = b3 * w[3];
        int r = r_lo;
        for (; r + 3 < r_hi; r += 4) {  // all loads of a trip before its stores
          float qv[4];
          float4 vb[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            qv[u] = A[(r + u) * ld + c];
            vb[u] = *reinterpret_cast<const float4*>(Vb + (r + u) * NBQ);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            qv[u] = fmaf(-vb[u].x, tw[0], qv[u]);
            qv[u] = fmaf(-vb[u].y, tw[1], qv[u]);
            qv[u] = fmaf(-vb[u].z, tw[2], qv[u]);
            qv[u] = fmaf(-vb[u].w, tw[3], qv[u]);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) A[(r + u) * ld + c] = qv[u];
        }
        for (; r < r_hi; ++r) {
          float qv = A[r * ld + c];
#pragma unroll
          for (int i = 0; i < NBQ; ++i) qv = fmaf(-Vb[r * NBQ + i], tw[i], qv);
          A[r * ld + c] = qv;
        }
      }
      bar_named(1, QT);
    }
    // first row and column of Q are e_0
    for (int i = qt; i < n; i += QT) {
      A[i * ld] = (i == 0) ? 1.f : 0.f;
      A[i] = (i == 0) ? 1.f : 0.f;
    }
    if (n == 2 && qt == 0) {  // no reflector at all: Q = I
      A[ld + 1] = 1.f;
    }
  }
  }

  // ---------------- eigenvalues of T by bisection ----------------
  // dv = diagonal, ev[i] couples i and i+1.  vv <- ev^2, pv <- eigenvalues (ascending).
  float* e2 = vv;
  float* lam = pv;
  float tnorm = 0.f;
  if (warp < nbw) {
    float lo = 3.0e38f, hi = -3.0e38f;
    for (int i = tid; i < n; i += ET) {
      const float el = (i > 0) ? fabsf(ev[i - 1]) : 0.f, er = (i + 1 < n) ? fabsf(ev[i]) : 0.f;
      lo = fminf(lo, dv[i] - el - er);
      hi = fmaxf(hi, dv[i] + el + er);
      e2[i] = ev[i] * ev[i];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if (lane == 0) {
      s_red[warp] = lo;
      s_sig[warp] = hi;
    }
    bar_named(2, ET);
    lo = s_red[0];
    hi = s_sig[0];
    for (int w = 1; w < nbw; ++w) {
      lo = fminf(lo, s_red[w]);
      hi = fmaxf(hi, s_sig[w]);
    }
    const float tn = fmaxf(fabsf(lo), fabsf(hi));
    lo -= 2.4e-7f * tn + 1e-30f;
    hi += 2.4e-7f * tn + 1e-30f;
    // Sturm count in product form on T / |T| (no division on the serial chain):
    //   p_0 = 1, p_1 = d_0 - x, p_{i+1} = (d_i - x) p_i - e_{i-1}^2 p_{i-1};
    // the number of sign changes along the sequence is the number of eigenvalues below x.
    // Both running values are rescaled together whenever they leave [1e-8, 1e8].
    const float itn = 1.0f / fmaxf(tn, 1e-30f);
    for (int i = tid; i < n; i += ET) {
      dn[i] = dv[i] * itn;
      e2[i] = e2[i] * itn * itn;
    }
    bar_named(2, ET);
    // the entries of two steps side by side, one 16-byte load per trip of the count below
    float4* tq = reinterpret_cast<float4*>(cs);
    const int ntrip = (n - 1) >> 1;
    for (int t = tid; t < ntrip; t += ET)
      tq[t] = make_float4(dn[2 * t + 1], e2[2 * t], dn[2 * t + 2], e2[2 * t + 1]);
    bar_named(2, ET);
    auto sturm = [&](float x) {
      // two steps per trip, and the pair is re-centred once per trip (entries can be as small as
      // rounding noise, 1e-7 of the largest, so it can shrink by 1e-14 in a trip: the thresholds
      // leave room).  A sign change is a difference of sign bits; a zero takes the sign of its
      // bit, which gives the same total because the value after it has the opposite sign of the
      // one before it.
      float p0 = 1.f, p1 = dn[0] - x;
      unsigned cnt = __float_as_uint(p1) >> 31;
      for (int t = 0; t < ntrip; ++t) {
        const float4 q = tq[t];
        const float pa = fmaf(q.x - x, p1, -q.y * p0);
        const float pb = fmaf(q.z - x, pa, -q.w * p1);
        cnt += ((__float_as_uint(pa) ^ __float_as_uint(p1)) >> 31) +
               ((__float_as_uint(pb) ^ __float_as_uint(pa)) >> 31);
        p0 = pa;
        p1 = pb;
        const float sc = fmaxf(fabsf(p0), fabsf(p1));
        if (sc < 1e-8f) {
          p0 *= 1e16f;
          p1 *= 1e16f;
        } else if (sc > 1e8f) {
          p0 *= 1e-16f;
          p1 *= 1e-16f;
        }
      }
      if (!(n & 1)) {  // one step left
        const float pa = fmaf(dn[n - 1] - x, p1, -e2[n - 2] * p0);
        cnt += (__float_as_uint(pa) ^ __float_as_uint(p1)) >> 31;
      }
      return (int)cnt;
    };
    const float lon = lo * itn, hin = hi * itn;
    // First round, shared by all eigenvalues: counts at n points spaced geometrically from the
    // top of the spectrum down to a little under the smallest eigenvalue that can pass the rank
    // cut-off.  Each eigenvalue starts its own bisection from the two points around it.
    int* gcnt = reinterpret_cast<int*>(pv);
    const float glo = fmaxf(0.06f * rank_tol * rank_tol, 1e-9f);
    const bool use_grid = hin > 2.0f * glo;
    const float lr = use_grid ? log2f(glo / hin) / (float)n : 0.f;
    auto grid = [&](int t) { return hin * exp2f(lr * (float)(n - t)); };
    if (use_grid) {
      if (tid < n) gcnt[tid] = sturm(grid(tid));
      bar_named(2, ET);
    }
    float a = lon, bhi = hin;
    if (use_grid && tid < n) {
      int tl = -1, th = n;  // the count is 0 at lon (t = -1) and n at hin (t = n)
      while (th - tl > 1) {
        const int mid = (tl + th) >> 1;
        if (gcnt[mid] > tid) th = mid; else tl = mid;
      }
      if (tl >= 0) a = fmaxf(lon, grid(tl));
      if (th < n) bhi = fminf(hin, grid(th));
    }
    bar_named(2, ET);  // the counts are overwritten by the eigenvalues below
    if (tid < n) {
      // eigenvalue number tid (0 = smallest): plain bisection, one thread per eigenvalue (the
      // counts are bound by instruction issue, so evaluating several points per round on
      // neighbouring lanes costs more than the rounds it saves)
      // An interval that lies wholly under the floor below which no eigenvector is computed
      // stops at a thousandth of that floor: such an eigenvalue only enters the energy check.
      const float floor_n = 0.25f * rank_tol * rank_tol;
      for (int it = 0; it < 48; ++it) {
        const float x = 0.5f * (a + bhi);
        if (!(x > a) || !(x < bhi)) break;
        if (bhi < floor_n && bhi - a < 1e-3f * floor_n) break;
        if (sturm(x) > tid) bhi = x; else a = x;
      }
      lam[tid] = 0.5f * (a + bhi) * tn;
    }
    tnorm = tn;
    bar_named(2, ET);
  }

  // ---------------- eigenvectors of T by inverse iteration ----------------
  const float keep_floor = 0.25f * rank_tol * rank_tol * tnorm;
  {
    const size_t img = (size_t)b * n * n;
    float* u0 = u0g + img;
    float* u1 = u1g + img;
    float* u2 = u2g + img;
    float* y = yg + img * nparts;
    float* ml = mlg + (size_t)b * ml_stride;
    if (tid < n) {
      const int t = tid;
      float x = lam[t];
      const bool wanted = x >= keep_floor;
      // an eigenvalue bisection could not tell from its lower neighbour is nudged up so the two
      // solves do not return the same vector
      const float sep = 1.2e-6f * fmaxf(fabsf(x), 1e-3f * tnorm);
      if (t > 0 && x - lam[t - 1] < sep) x = lam[t - 1] + sep * (float)(1 + (t & 3));
      const float tiny = fmaxf(tnorm, 1e-30f) * 1.1920929e-7f;
      if (wanted) {
        // factor T - x I once, with row interchanges (|multiplier| <= 1).  Stored per row: the
        // reciprocal pivot, the two entries right of it, and the multiplier, to which 4 is
        // added when the rows were swapped.
        {
          float a = dv[0] - x, bb = (n > 1) ? ev[0] : 0.f, c = 0.f;
          for (int i = 0; i + 1 < n; ++i) {
            const float sub = ev[i], dnx = dv[i + 1] - x, en = (i + 2 < n) ? ev[i + 1] : 0.f;
            const bool sw = fabsf(a) < fabsf(sub);
            float piv = sw ? sub : a;
            const float oth = sw ? a : sub;
            if (fabsf(piv) < tiny) piv = copysignf(tiny, piv);
            const float rp = 1.0f / piv;
            const float mlt = oth * rp;
            const float p1 = sw ? dnx : bb, p2 = sw ? en : c;
            const float q1 = sw ? bb : dnx, q2 = sw ? c : en;
            u0[(size_t)i * n + t] = rp;
            u1[(size_t)i * n + t] = p1;
            u2[(size_t)i * n + t] = p2;
            ml[(size_t)i * n + t] = sw ? mlt + 4.0f : mlt;
            a = fmaf(-mlt, p1, q1);
            bb = fmaf(-mlt, p2, q2);
            c = 0.f;
          }
          if (fabsf(a) < tiny) a = copysignf(tiny, a);
          u0[(size_t)(n - 1) * n + t] = 1.0f / a;
          u1[(size_t)(n - 1) * n + t] = 0.f;
          u2[(size_t)(n - 1) * n + t] = 0.f;
        }
        float scale = 1.f, nrm = 0.f;
        for (int it = 0; it < 3; ++it) {
          if (it > 0) {
            // apply the elimination to the right-hand side (the previous solution, rescaled)
            float cur = y[t] * scale;
            for (int i0 = 0; i0 + 1 < n; i0 += 8) {
              float nx[8], me[8];
#pragma unroll
              for (int u = 0; u < 8; ++u)
                if (i0 + u + 1 < n) {
                  nx[u] = y[(size_t)(i0 + u + 1) * n + t] * scale;
                  me[u] = ml[(size_t)(i0 + u) * n + t];
                }
#pragma unroll
              for (int u = 0; u < 8; ++u) {
                const int i = i0 + u;
                if (i + 1 < n) {
                  const bool sw = me[u] > 2.0f;
                  const float mlt = sw ? me[u] - 4.0f : me[u];
                  const float hi_ = sw ? nx[u] : cur, lo_ = sw ? cur : nx[u];
                  y[(size_t)i * n + t] = hi_;
                  cur = fmaf(-mlt, hi_, lo_);
                }
              }
            }
            y[(size_t)(n - 1) * n + t] = cur;
          }
          // back substitution (first pass: right-hand side of ones), eight rows per group of loads
          float y1 = 0.f, y2 = 0.f, big = 0.f;
          nrm = 0.f;
          for (int i1 = n - 1; i1 >= 0; i1 -= 8) {
            float rh[8], p0[8], p1[8], p2[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int i = i1 - u;
              if (i >= 0) {
                rh[u] = (it == 0) ? 1.f : y[(size_t)i * n + t];
                p0[u] = u0[(size_t)i * n + t];
                p1[u] = u1[(size_t)i * n + t];
                p2[u] = u2[(size_t)i * n + t];
              }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int i = i1 - u;
              if (i >= 0) {
                const float yi = (rh[u] - p1[u] * y1 - p2[u] * y2) * p0[u];
                y[(size_t)i * n + t] = yi;
                big = fmaxf(big, fabsf(yi));
                nrm = fmaf(yi, yi, nrm);
                y2 = y1;
                y1 = yi;
              }
            }
          }
          scale = 1.0f / fmaxf(big, 1e-30f);  // keeps the next right-hand side in range
        }
        {
          // normalise; Rayleigh quotient on T
          const float inv = rsqrtf(fmaxf(nrm * scale * scale, 1e-30f)) * scale;
          float rq = 0.f, prev = 0.f;
          for (int i0 = 0; i0 < n; i0 += 8) {
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
              if (i0 + u < n) v[u] = y[(size_t)(i0 + u) * n + t] * inv;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int i = i0 + u;
              if (i < n) {
                y[(size_t)i * n + t] = v[u];
                rq = fmaf(dv[i] * v[u], v[u], rq);
                if (i > 0) rq = fmaf(2.0f * ev[i - 1] * prev, v[u], rq);
                prev = v[u];
              }
            }
          }
          e2[t] = rq;  // e2 is free after the bisection
        }
      } else {
        for (int i = 0; i < n; ++i) y[(size_t)i * n + t] = 0.f;
        e2[t] = lam[t];
      }
    }
    __syncthreads();
    for (int p = tid; p < n; p += 512) theta[(size_t)b * n + p] = fmaxf(e2[p], 0.f);
    if (emit_factors) {
      float* QT = ZTg + img;
      for (int e = tid; e < n * n; e += 512) {
        const int j = e / n, i = e - j * n;
        QT[e] = A[i * ld + j];
      }
      __syncthreads();
      for (int e = tid; e < n * n; e += 512) {   // Y through shared memory, to turn it over
        const int j = e / n, p = e - j * n;
        A[j * ld + p] = __ldcg(y + e);
      }
      __syncthreads();
      float* YT = u0;  // the factorisations kept there are no longer needed
      for (int e = tid; e < n * n; e += 512) {
        const int p = e / n, j = e - p * n;
        YT[e] = A[j * ld + p];
      }
      if (tid == 0 && s_fail) atomicMax(&status[b], (int)TC_ERR_NOT_CONVERGED);
      return;
    }
    // ---------------- Z = Q Y:  ZT[p][i] = sum_j Q[i][j] Y[j][p] ----------------
    // thread = (four eigenvectors p, twelve rows i): per j one 16-byte load of Y (coalesced over
    // p) and twelve broadcast reads of Q from shared memory feed 48 multiply-adds
    float* out = ZTg + img;
    const bool vec = (n & 3) == 0;
    const int npg = (n + 3) >> 2, nrg = (n + 11) / 12;
    for (int w = tid; w < npg * nrg; w += 512) {
      const int rg = w / npg, pg = w - rg * npg;
      const int p0 = pg * 4, i0 = rg * 12;
      float acc[12][4];
      const float* qrow[12];
#pragma unroll
      for (int u = 0; u < 12; ++u) {
        qrow[u] = A + min(i0 + u, n - 1) * ld;  // rows past the end are computed and dropped
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = 0.f;
      }
#pragma unroll 4
      for (int j = 0; j < n; ++j) {
        float4 yv;
        const float* yr = y + (size_t)j * n + p0;
        if (vec) {
          yv = __ldcg(reinterpret_cast<const float4*>(yr));
        } else {
          yv.x = __ldcg(yr);
          yv.y = (p0 + 1 < n) ? __ldcg(yr + 1) : 0.f;
          yv.z = (p0 + 2 < n) ? __ldcg(yr + 2) : 0.f;
          yv.w = (p0 + 3 < n) ? __ldcg(yr + 3) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 12; ++u) {
          const float a = qrow[u][j];
          acc[u][0] = fmaf(a, yv.x, acc[u][0]);
          acc[u][1] = fmaf(a, yv.y, acc[u][1]);
          acc[u][2] = fmaf(a, yv.z, acc[u][2]);
          acc[u][3] = fmaf(a, yv.w, acc[u][3]);
        }
      }
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        if (p0 + v >= n) continue;
        float* orow = out + (size_t)(p0 + v) * n + i0;
        if (vec && i0 + 12 <= n) {
#pragma unroll
          for (int u = 0; u < 12; u += 4)
            *reinterpret_cast<float4*>(orow + u) =
                make_float4(acc[u][v], acc[u + 1][v], acc[u + 2][v], acc[u + 3][v]);
        } else {
#pragma unroll
          for (int u = 0; u < 12; ++u)
            if (i0 + u < n) orow[u] = acc[u][v];
        }
      }
    }
  }
  if (tid == 0 && s_fail) atomicMax(&status[b], (int)TC_ERR_NOT_CONVERGED);
}

typedef void (*jacobi_fn)(const float*, float*, float*, float*, int, int, float, int, int32_t*, float, float);

static jacobi_fn pick_jacobi(int n) {
  const int r = (n + 31) / 32;
  if (r <= 1) return jacobi_kernel<1>;
  if (r <= 2) return jacobi_kernel<2>;
  if (r <= 3) return jacobi_kernel<3>;
  if (r <= 4) return jacobi_kernel<4>;
  if (r <= 5) return jacobi_kernel<5>;
  if (r <= 6) return jacobi_kernel<6>;
  if (r <= 8) return jacobi_kernel<8>;
  if (r <= 10) return jacobi_kernel<10>;
  if (r <= 14) return jacobi_kernel<14>;
  if (r <= 18) return jacobi_kernel<18>;
  if (r <= 24) return jacobi_kernel<24>;
  if (r <= 32) return jacobi_kernel<32>;
  return nullptr;
}

constexpr size_t SMEM_LIMIT = 220 * 1024;  // leaves room for the static shared variables

static void launch_jacobi(const float* H, float* W, float* ZT, float* theta, int n, int batch,
                          int max_sweeps, float rank_tol, float* scr1, float* scr2, float* scr3,
                          float* scr4, size_t scr4_stride, int32_t* status, cudaStream_t st,
                          int nparts = 1, int emit_factors = 0) {
  Scope scope_(KC_JACOBI, st);
  {
    const size_t tri = ((size_t)n * (n | 1) + 27 * (size_t)((n + 3) & ~3)) * sizeof(float);
    if (n >= 3 && tri <= SMEM_LIMIT && scr1 != nullptr) {
      auto go = [&](auto kernel) {
        cudaFuncSetAttribute((const void*)kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tri);
        { kernel<<<batch, 512, tri, st>>>(H, ZT, theta, n, rank_tol, W, scr1, scr2, scr3, scr4, scr4_stride, status, nparts, emit_factors); note_launch(); }
      };
      switch (n) {
        case 128: go(tridiag_eig_kernel<128>); break;
        case 144: go(tridiag_eig_kernel<144>); break;
        case 160: go(tridiag_eig_kernel<160>); break;
        case 192: go(tridiag_eig_kernel<192>); break;
        default: go(tridiag_eig_kernel<0>); break;
      }
      return;
    }
  }
  jacobi_fn fn = pick_jacobi(n);
  const size_t need = 2 * (size_t)n * n * sizeof(float);
  const int use_smem = need <= SMEM_LIMIT;
  const size_t smem = use_smem ? need : 0;
  if (use_smem) cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  // off-diagonal threshold a little above the rounding noise of a length-n float32 dot product
  const float tol = fmaxf(1e-6f, 2.5f * sqrtf((float)n) * 1.1920929e-7f);
  // Eigenvalue floors, relative to the largest diagonal entry.  Column pairs that are both
  // under the float32 rounding level of that entry are never rotated; rotations between two
  // columns that are both under the eigenvalue rank_tol cuts at are done but do not count
  // towards "this sweep still rotated".
  const float floor_rel = 1e-6f;
  const float count_rel = fmaxf(floor_rel, rank_tol * rank_tol);
  { fn<<<batch, 512, smem, st>>>(H, W, ZT, theta, n, max_sweeps, tol, use_smem, status, floor_rel, count_rel); note_launch(); }
}

static void launch_chol_inv(const float* S, float* RinvT, float* Rwork, int k, int batch,
                            float shift_rel, int32_t* status, cudaStream_t st, int nparts) {
  Scope scope_(KC_CHOL, st);
  const size_t fast = ((size_t)k * (k | 1) + 2 * (size_t)CNB * k + (size_t)(k / CNB) * CNB * CNB) * sizeof(float);
  if (k % CNB == 0 && k >= CNB && fast <= SMEM_LIMIT) {
    auto go = [&](auto kernel) {
      cudaFuncSetAttribute((const void*)kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fast);
      { kernel<<<batch, 512, fast, st>>>(S, RinvT, k, shift_rel, status, nparts); note_launch(); }
    };
    switch (k) {
      case 128: go(chol_inv_fast_kernel<128>); break;
      case 144: go(chol_inv_fast_kernel<144>); break;
      case 160: go(chol_inv_fast_kernel<160>); break;
      case 192: go(chol_inv_fast_kernel<192>); break;
      default: go(chol_inv_fast_kernel<0>); break;
    }
    return;
  }
  const size_t blocked = (size_t)k * (k | 1) * sizeof(float);
  // (the blocked kernel keeps 2 x 4 outputs per thread in registers in its last step)
  if (blocked <= SMEM_LIMIT && (size_t)k * (CNB / 4) <= 2 * 512) {
    cudaFuncSetAttribute((const void*)chol_inv_blocked_kernel,
                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)blocked);
    { chol_inv_blocked_kernel<<<batch, 512, blocked, st>>>(S, RinvT, k, shift_rel, status, nparts); note_launch(); }
    return;
  }
  const size_t need = 2 * (size_t)k * k * sizeof(float);
  const int use_smem = need <= SMEM_LIMIT;
  const size_t smem = use_smem ? need : 0;
  if (use_smem)
    cudaFuncSetAttribute((const void*)chol_inv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  { chol_inv_kernel<<<batch, 512, smem, st>>>(S, RinvT, Rwork, k, shift_rel, use_smem, status); note_launch(); }
}

// ==========================================================================================
// out [C][R] = in [R][C]^T per image, 32 x 32 tiles through shared memory.
// grid (C tiles, R tiles, batch), block (32, 8).
// ==========================================================================================
__global__ void __launch_bounds__(256) transpose_kernel(const float* __restrict__ in, int R, int C,
                                                       float* __restrict__ out) {
  __shared__ float t[32][33];
  const int b = blockIdx.z, r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
  const size_t RC = (size_t)R * C;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = r0 + ty + 8 * i, c = c0 + tx;
    t[ty + 8 * i][tx] = (r < R && c < C) ? in[(size_t)b * RC + (size_t)r * C + c] : 0.f;
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int c = c0 + ty + 8 * i, r = r0 + tx;
    if (r < R && c < C) out[(size_t)b * RC + (size_t)c * R + r] = t[tx][ty + 8 * i];
  }
}

static void launch_transpose(const float* in, int R, int C, int batch, float* out, cudaStream_t st, int cls) {
  Scope scope_(cls, st);
  dim3 grid((C + 31) / 32, (R + 31) / 32, batch), block(32, 8);
  { transpose_kernel<<<grid, block, 0, st>>>(in, R, C, out); note_launch(); }
}

// ==========================================================================================
// Eq. 3-6 and the outputs that go with it.  One block per image.
//   theta [k]   eigenvalues of G (unsorted);  sigma_i = sqrt(theta_i)
//   PT [k][N]   PT[p][x] = component of token x along eigenvector p (u_xp)
//   C(x) = sum over p with sigma_p > rank_tol * sigma_max of |u_xp| sigma_p
// ==========================================================================================
__global__ void __launch_bounds__(256) ics_kernel(const float* __restrict__ theta,
                                                 const float* __restrict__ PT, float* __restrict__ C,
                                                 float* __restrict__ sigma_sorted,
                                                 int32_t* __restrict__ rank_out,
                                                 int32_t* __restrict__ status, int N, int k, int q,
                                                 float rank_tol, int full,
                                                 const float* __restrict__ G) {
  // G (subspace solve only): the Gram matrix, for the energy check below
  // grid (token chunks of 64, images): every block ranks the k singular values again (k^2
  // comparisons, cheap) and sums Eq. 3-6 for its own tokens, four threads to a token (each a
  // quarter of the range of p, its loads in flight together); chunk 0 writes sigma and the rank.
  extern __shared__ float sig[];  // [k] sigma, then [k] weights (sigma or 0)
  float* wgt = sig + k;
  __shared__ float s_red[8];
  __shared__ int s_cnt[8];
  __shared__ float s_part[4][64];
  const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool writer = blockIdx.x == 0;
  float mx = 0.f;
  for (int p = tid; p < k; p += 256) {
    const float s = sqrtf(fmaxf(theta[(size_t)b * k + p], 0.f));
    sig[p] = s;
    mx = fmaxf(mx, s);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) s_red[warp] = mx;
  __syncthreads();
  float smax = s_red[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) smax = fmaxf(smax, s_red[w]);
  const float cut = rank_tol * smax;
  // O has at most q = min(N, d) non-zero singular values: only the q largest eigenvalues of G
  // can be one, whatever rounding left in the others.
  int cnt = 0;
  for (int p = tid; p < k; p += 256) {
    const float s = sig[p];
    int pos = 0;
    for (int o = 0; o < k; ++o) pos += (sig[o] > s) || (sig[o] == s && o < p);
    const bool on = (s > cut) && (pos < q);
    wgt[p] = on ? s : 0.f;
    cnt += on;
    if (writer && sigma_sorted && pos < q) sigma_sorted[(size_t)b * q + pos] = s;
  }
  if (writer && sigma_sorted)
    for (int p = k + tid; p < q; p += 256) sigma_sorted[(size_t)b * q + p] = 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  if (lane == 0) s_cnt[warp] = cnt;
  __syncthreads();
  if (writer && tid == 0) {
    int r = 0;
    for (int w = 0; w < 8; ++w) r += s_cnt[w];
    if (rank_out) rank_out[b] = r;
    if (!full && r > k - 8) atomicMax(&status[b], (int)TC_ERR_RANK_CAP);
  }
  if (writer && !full && G != nullptr && warp == 0) {
    // What the subspace did not capture: trace(G) - sum(theta) is the energy of O outside it.
    // If the directions left out were all under the rank cut-off, that is at most
    // (q - k) (rank_tol sigma_1)^2; more means a direction above the cut-off was missed (a
    // rank above the hint that the count above could not see), and Eq. 3-6 would be truncated.
    float tr = 0.f, st = 0.f;
    const float* Gb = G + (size_t)b * N * N;
    for (int x0 = 0; x0 < N; x0 += 256) {  // eight loads in flight
      float dgl[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int x = x0 + u * 32 + lane;
        dgl[u] = (x < N) ? Gb[(size_t)x * N + x] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) tr += dgl[u];
    }
    for (int p = lane; p < k; p += 32) st += sig[p] * sig[p];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      tr += __shfl_xor_sync(0xffffffffu, tr, o);
      st += __shfl_xor_sync(0xffffffffu, st, o);
    }
    const float allow = (float)max(q - k, 0) * cut * cut + 1e-5f * tr;
    if (lane == 0 && tr - st > allow) atomicMax(&status[b], (int)TC_ERR_RANK_CAP);
  }
  const float* PTb = PT + (size_t)b * k * N;
  const int xl = tid & 63, part = tid >> 6;
  const int x = blockIdx.x * 64 + xl;
  const int per = (k + 3) >> 2;
  const int p_lo = part * per, p_hi = min(k, p_lo + per);
  float acc = 0.f;
  if (x < N) {
    // terms of a quarter in the order p = p_lo, p_lo + 1, ...; twelve loads in flight
    int p = p_lo;
    for (; p + 11 < p_hi; p += 12) {
      float v[12];
#pragma unroll
      for (int u = 0; u < 12; ++u) v[u] = PTb[(size_t)(p + u) * N + x];
#pragma unroll
      for (int u = 0; u < 12; ++u) acc = fmaf(fabsf(v[u]), wgt[p + u], acc);
    }
    for (; p < p_hi; ++p) acc = fmaf(fabsf(PTb[(size_t)p * N + x]), wgt[p], acc);
  }
  s_part[part][xl] = acc;
  __syncthreads();
  if (part == 0 && x < N)
    C[(size_t)b * N + x] = (s_part[0][xl] + s_part[1][xl]) + (s_part[2][xl] + s_part[3][xl]);
}

__global__ void fill_i32_kernel(int32_t* p, int n, int v) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

void fill_i32(int32_t* p, int n, int v, cudaStream_t st) {
  Scope scope_(KC_FILL, st);
  { fill_i32_kernel<<<(n + 255) / 256, 256, 0, st>>>(p, n, v); note_launch(); }
}

// ==========================================================================================
// The whole of Eq. 3-5 / 3-6 for a batch, given G in the workspace.
// ==========================================================================================
tc_status launch_ics(const Dims& D, const Plan& P, char* ws, int b0, const void* O, float* C_out,
                     float* sigma_out, int32_t* rank_out, int32_t* img_status, cudaStream_t st,
                     float* full_scratch, cudaEvent_t g_ready) {
  // D.B images starting at image b0 of the workspace arrays; O and the outputs already point at
  // image b0.
  const int B = D.B, N = D.N, k = D.k;
  const int q = min(D.N, D.d);
  const size_t sG = (size_t)N * N, sY = (size_t)N * k, sK = (size_t)k * k;
  float* G = (float*)(ws + P.G) + b0 * sG;
  float* W = (float*)(ws + P.W) + b0 * sK;
  float* ZT = (float*)(ws + P.ZT) + b0 * sK;
  float* theta = (float*)(ws + P.sigma) + (size_t)b0 * k;

  if (D.full) {
    if (g_ready) cudaStreamWaitEvent(st, g_ready, 0);
    // with scratch for it (four N x N arrays per image) the tridiagonal solver takes the full
    // problem when it fits in shared memory: it has no sweeps that a spectrum without a gap at
    // the rounding level could keep alive
    float* fs = full_scratch;
    launch_jacobi(G, W, ZT, theta, N, B, D.max_sweeps, D.rank_tol, fs, fs ? fs + (size_t)B * sG : nullptr,
                  fs ? fs + 2 * (size_t)B * sG : nullptr, fs ? fs + 3 * (size_t)B * sG : nullptr, sG,
                  img_status, st);
    Scope scope_(KC_ICS, st);
    { ics_kernel<<<dim3((N + 63) / 64, B), 256, 2 * (size_t)N * sizeof(float), st>>>(
          theta, ZT, C_out, sigma_out, rank_out, img_status, N, N, q, D.rank_tol, 1, nullptr); note_launch(); }
    return TC_OK;
  }
  auto sketch_into = [&](float* Y0) {
    Scope scope_(KC_SKETCH, st);
    const int L = 16 / D.esz;
    if (k % L == 0 && k / L <= 256 && (size_t)D.d * sizeof(float) <= 48 * 1024) {
      const int kg = k / L;
      const int rows = max(1, 256 / kg);
      dim3 block(kg, rows), grid((N + rows - 1) / rows, B);
      const size_t smem = (size_t)D.d * sizeof(float);
      TC_WITH_STORAGE_TYPE(D,
        sketch_vec_kernel<T, 16 / sizeof(T)><<<grid, block, smem, st>>>((const T*)O, Y0, N, D.d, k);
        note_launch(););
    } else {
      dim3 grid(N, B);
      const int threads = (k + 31) / 32 * 32;
      TC_WITH_STORAGE_TYPE(D,
        sketch_kernel<T><<<grid, threads, 0, st>>>((const T*)O, Y0, N, D.d, k);
        note_launch(););
    }
  };
  if (D.tcp) {
    // ---- the products on the tensor cores (gemm_f32x3.cu: C = A B^T, both operands with the
    //      contraction index contiguous).  Every tall panel is therefore kept twice, row-major
    //      [N][k] and transposed [k][N]; a product writes whichever forms its consumers read.
    float* Ar = (float*)(ws + P.PA) + b0 * sY;
    float* At = (float*)(ws + P.PA) + (size_t)P.panel_T_off / sizeof(float) + b0 * sY;
    float* Br = (float*)(ws + P.PB) + b0 * sY;
    float* Bt = (float*)(ws + P.PB) + (size_t)P.panel_T_off / sizeof(float) + b0 * sY;
    float* Sk = (float*)(ws + P.Sk) + b0 * sK;
    float* Hk = (float*)(ws + P.Hk) + b0 * sK;
    float* Rinv = (float*)(ws + P.Rinv) + b0 * sK;
    float* Es = (float*)(ws + P.Es) + b0 * 4 * sK;
    int32_t* stp = img_status;
    tc_status err = TC_OK;
    auto mm = [&](const float* A_, const float* B_, int M_, int K_, float* c, float* ct, int cls) {
      if (err == TC_OK) err = launch_gemm_f32x3(A_, B_, M_, k, K_, B, c, ct, stp, st, cls);
    };
    // one Cholesky-QR pass  dst = src R^{-1}  with  R^T R = src^T src + shift
    auto pass = [&](const float* srcR, const float* srcT, float* dstR, float* dstT, float shift_rel) {
      mm(srcT, srcT, k, N, Sk, nullptr, KC_GEMM_TN);
      if (err != TC_OK) return;
      launch_chol_inv(Sk, Rinv, nullptr, k, B, shift_rel, stp, st, 1);
      mm(srcR, Rinv, N, k, dstR, dstT, KC_GEMM);   // Rinv holds R^{-T}: (Y R^{-1})[x][c] = Y[x][:] . Rinv[c][:]
    };
    // 1. sketch of the column space of O, in both forms
    sketch_into(Ar);
    launch_transpose(Ar, N, k, B, At, st, KC_SKETCH);
    // 2. a well-conditioned basis Q0 of the sketch (only its transposed form is read)
    pass(Ar, At, nullptr, Bt, 1e-6f);
    // 3. Y1 = G Q0, then two passes: the first (shifted) brings the condition number from ~1e7
    //    down to ~1e3, the second leaves a basis whose departure from orthonormality lies in the
    //    directions under the rank cut-off; the Ritz values above it are unaffected
    if (g_ready) cudaStreamWaitEvent(st, g_ready, 0);
    mm(G, Bt, N, N, Ar, At, KC_GEMM_GQ);
    pass(Ar, At, Br, Bt, 1e-6f);
    pass(Br, Bt, Ar, At, 1e-7f);  // Q1 in set A
    // 4. Rayleigh-Ritz:  T = G Q1 (kept transposed),  H = Q1^T T
    mm(G, At, N, N, nullptr, Bt, KC_GEMM_GQ);
    mm(At, Bt, k, N, Hk, nullptr, KC_GEMM_TN);
    if (err != TC_OK) return err;
    // The solver leaves the eigenvectors of H as the two factors Z = Q Y (Q from the reduction
    // to tridiagonal form, Y the eigenvectors of the tridiagonal matrix): Q^T in QTk, Y^T in YTk.
    float* QTk = Sk;  // the k x k matrices of the passes are free now
    float* YTk = Es;  // (the solver's first work array, handed back as Y^T)
    launch_jacobi(Hk, Es, QTk, theta, k, B, D.max_sweeps, D.rank_tol, Es + (size_t)B * sK,
                  Es + 2 * (size_t)B * sK, Rinv, Es + 3 * (size_t)B * sK, sK, stp, st, 1, 1);
    // 5. eigenvectors of G in the subspace, U = Q1 Q Y, as two products:
    //    W = Q1 Q, then PT[p][x] = sum_j Y[j][p] W[x][j] (W Y written transposed)
    mm(Ar, QTk, N, k, Br, nullptr, KC_GEMM);
    float* PT = Bt;
    mm(Br, YTk, N, k, nullptr, PT, KC_GEMM);
    if (err != TC_OK) return err;
    Scope scope_(KC_ICS, st);
    { ics_kernel<<<dim3((N + 63) / 64, B), 256, 2 * (size_t)k * sizeof(float), st>>>(
          theta, PT, C_out, sigma_out, rank_out, img_status, N, k, q, D.rank_tol, 0, G); note_launch(); }
    return TC_OK;
  }
  float* Y0 = (float*)(ws + P.Y0) + b0 * sY;
  float* Y1 = (float*)(ws + P.Y1) + b0 * sY;
  float* Y2 = (float*)(ws + P.Y2) + b0 * sY;
  const int parts = tn_parts(k);  // the k x k products come in this many parts per image
  float* Sm = (float*)(ws + P.Sm) + b0 * sK * parts;
  float* Rinv = (float*)(ws + P.Rinv) + b0 * sK;
  float* Hm = (float*)(ws + P.Hm) + b0 * sK * parts;

  // 1. sketch of the column space of O
  sketch_into(Y0);
  // one Cholesky-QR pass: dst = src R^{-1},  R^T R = src^T src (+ shift)
  auto cholqr_pass = [&](const float* src, float* dst, float shift_rel) {
    gemm_tn_sym(src, src, Sm, k, N, sY, sY, B, st, KC_GEMM_TN);
    launch_chol_inv(Sm, Rinv, W, k, B, shift_rel, img_status, st, parts);
    gemm<float, float, false, true>(src, Rinv, dst, N, k, k, k, k, k, sY, sK, sY, B, st, KC_GEMM, GEMM_B_UPPER);
  };
  const float kShift = 1e-6f;
  // 2. a well-conditioned (not orthonormal) basis Q0 of the sketch: one shifted pass takes the
  //    condition number from ~1e3 to a few units, which is all the next product needs
  cholqr_pass(Y0, Y1, kShift);
  { float* t = Y0; Y0 = Y1; Y1 = t; }  // Q0 in Y0
  // 3. one multiplication by G sharpens the subspace:  Y1 = G Q0, then orthonormalise
  if (g_ready) cudaStreamWaitEvent(st, g_ready, 0);
  gemm<float, float, false, false>(G, Y0, Y1, N, k, N, N, k, k, sG, sY, sY, B, st, KC_GEMM_GQ);
  cholqr_pass(Y1, Y2, kShift);
  cholqr_pass(Y2, Y1, kShift);
  cholqr_pass(Y1, Y2, 0.f);  // Q1 in Y2
  // 4. Rayleigh-Ritz:  H = Q1^T G Q1
  gemm<float, float, false, false>(G, Y2, Y1, N, k, N, N, k, k, sG, sY, sY, B, st, KC_GEMM_GQ);   // T = G Q1
  gemm_tn_sym(Y2, Y1, Hm, k, N, sY, sY, B, st, KC_GEMM_TN);   // H = Q1^T T (symmetric)
  // scratch of the solver: W, Sm, Rinv, Hm (k x k each) and the first k x k of each image's Y1 panel
  launch_jacobi(Hm, W, ZT, theta, k, B, D.max_sweeps, D.rank_tol, Sm, Rinv, Hm, Y1, sY, img_status, st, parts);
  // 5. eigenvectors of G restricted to the subspace:  PT[p][x] = sum_i ZT[p][i] Q1[x][i]
  gemm<float, float, false, true>(ZT, Y2, Y0, k, N, k, k, k, N, sK, sY, sY, B, st);
  Scope scope_(KC_ICS, st);
  { ics_kernel<<<dim3((N + 63) / 64, B), 256, 2 * (size_t)k * sizeof(float), st>>>(
        theta, Y0, C_out, sigma_out, rank_out, img_status, N, k, q, D.rank_tol, 0, G); note_launch(); }
  return TC_OK;
}

}  // namespace tc
