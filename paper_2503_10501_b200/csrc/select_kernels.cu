// Selection kernels: Stage I prune and the Set A / Set B split (Sec. 3.3.1 end, Eq. 3-9), the
// best-match search of Eq. 3-10, and the choice of the merged tokens (Sec. 3.3.2 end).
// Every selection is an exact radix select on the float bit patterns; ties go to the lower
// token index, so results are deterministic and independent of thread scheduling.
#include "tc_internal.cuh"

namespace tc {

constexpr int SEL_THREADS = 256;

// float -> uint32 whose unsigned order equals the float order (-0 < +0 is harmless here).
__device__ inline uint32_t orderable(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive prefix sum over the threads of a 256-thread block (thread order), total in *total.
__device__ int block_excl_scan(int v, int* sh /* >= 9 ints */, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();  // sh may still be read from a previous call
  if (lane == 31) sh[warp] = inc;
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    for (int w = 0; w < SEL_THREADS / 32; ++w) {
      int t = sh[w];
      sh[w] = run;
      run += t;
    }
    sh[8] = run;
  }
  __syncthreads();
  const int res = sh[warp] + inc - v;
  *total = sh[8];
  return res;
}

// k-th largest key (k in 1..n) of keys[0..n): returns the key value `thr` and how many of the
// keys equal to thr belong to the top k (`need_eq` >= 1).  MSB-first, 8 bits per pass; the bin
// that holds the k-th key is found by a block-wide scan of the histogram from the top bin down
// (thread t holds bin 255 - t), not by one thread walking it.
__device__ void block_select_kth(const uint32_t* keys, int n, int kth, int* hist /*256*/,
                                 uint32_t* sh_u /*2*/, int* sh_scan /*9*/, uint32_t* thr,
                                 int* need_eq) {
  uint32_t prefix = 0, mask = 0;
  int remaining = kth;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = threadIdx.x; i < 256; i += SEL_THREADS) hist[i] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += SEL_THREADS) {
      const uint32_t kx = keys[i];
      if ((kx & mask) == prefix) atomicAdd(&hist[(kx >> shift) & 255u], 1);
    }
    __syncthreads();
    const int mine = hist[255 - threadIdx.x];
    int tot;
    const int above = block_excl_scan(mine, sh_scan, &tot);  // keys in higher bins
    if (above < remaining && above + mine >= remaining) {      // exactly one thread
      sh_u[0] = 255u - threadIdx.x;
      sh_u[1] = (uint32_t)(remaining - above);
    }
    __syncthreads();
    prefix |= sh_u[0] << shift;
    mask |= 255u << shift;
    remaining = (int)sh_u[1];
    __syncthreads();
  }
  *thr = prefix;
  *need_eq = remaining;
}

// ------------------------------------------------------------------------------------------
// Stage I prune + Eq. 3-9.  One block per image.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(SEL_THREADS) prune_kernel(const float* __restrict__ E,
                                                           int32_t* __restrict__ setA,
                                                           int32_t* __restrict__ setB, int N,
                                                           int P, int nA, int nB) {
  extern __shared__ uint32_t keys[];  // [N]
  __shared__ int hist[256];
  __shared__ uint32_t sh_u[2];
  __shared__ int sh_scan[9];
  const int b = blockIdx.x;
  for (int i = threadIdx.x; i < N; i += SEL_THREADS) keys[i] = orderable(E[(size_t)b * N + i]);
  __syncthreads();
  uint32_t thrP, thrA = 0xffffffffu;
  int needP, needA = 0;
  block_select_kth(keys, N, P, hist, sh_u, sh_scan, &thrP, &needP);
  if (nA > 0) block_select_kth(keys, N, nA, hist, sh_u, sh_scan, &thrA, &needA);

  const int chunk = (N + SEL_THREADS - 1) / SEL_THREADS;
  const int i0 = min(N, (int)threadIdx.x * chunk), i1 = min(N, i0 + chunk);
  int eqP = 0, eqA = 0;
  for (int i = i0; i < i1; ++i) {
    eqP += (keys[i] == thrP);
    eqA += (keys[i] == thrA);
  }
  int tot;
  int eP = block_excl_scan(eqP, sh_scan, &tot);
  int eA = block_excl_scan(eqA, sh_scan, &tot);
  // classify this thread's tokens, count, then write in ascending order
  int cA = 0, cB = 0;
  uint32_t cls = 0;  // 2 bits per token of the chunk (chunk <= 16)
  for (int i = i0; i < i1; ++i) {
    const uint32_t kx = keys[i];
    bool inP = kx > thrP;
    if (kx == thrP) inP = (eP++ < needP);
    bool inA = (nA > 0) && (kx > thrA);
    if (nA > 0 && kx == thrA) inA = (eA++ < needA);
    const uint32_t c = inA ? 1u : (inP ? 2u : 0u);
    cls |= c << (2 * (i - i0));
    cA += (c == 1u);
    cB += (c == 2u);
  }
  int oA = block_excl_scan(cA, sh_scan, &tot);
  int oB = block_excl_scan(cB, sh_scan, &tot);
  for (int i = i0; i < i1; ++i) {
    const uint32_t c = (cls >> (2 * (i - i0))) & 3u;
    if (c == 1u) setA[(size_t)b * nA + oA++] = i;
    if (c == 2u) setB[(size_t)b * nB + oB++] = i;
  }
}

void launch_prune(const Dims& D, const float* E, int32_t* setA, int32_t* setB, cudaStream_t st) {
  Scope scope_(KC_PRUNE, st);
  { prune_kernel<<<D.B, SEL_THREADS, (size_t)D.N * sizeof(uint32_t), st>>>(E, setA, setB, D.N, D.P,
                                                                       D.nA, D.nB); note_launch(); }
}

// ------------------------------------------------------------------------------------------
// Eq. 3-10 from the Gram matrix:  cos(b, a) = G_ba / (max(|O_b|,1e-12) max(|O_a|,1e-12)).
// One warp per Set-B token; the lanes walk Set A.  Ties go to the lower token index.
// ------------------------------------------------------------------------------------------
__device__ inline float inv_norm_from_sq(float g) { return 1.0f / fmaxf(sqrtf(fmaxf(g, 0.f)), 1e-12f); }

__device__ inline void warp_best(float& val, int& idx) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, val, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    if (ov > val || (ov == val && oi < idx)) {
      val = ov;
      idx = oi;
    }
  }
}

__global__ void __launch_bounds__(128) match_gram_kernel(const float* __restrict__ G,
                                                        const int32_t* __restrict__ setA,
                                                        const int32_t* __restrict__ setB,
                                                        float* __restrict__ best_val,
                                                        int32_t* __restrict__ best_dst, int N,
                                                        int nA, int nB,
                                                        int32_t* __restrict__ status) {
  const int b = blockIdx.y;
  const int jb = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (jb >= nB) return;
  const float* Gb = G + (size_t)b * N * N;
  const int tb = setB[(size_t)b * nB + jb];
  // a token number outside [0, N) in a caller's list is reported and never used as an address
  if (tb < 0 || tb >= N) {
    if (lane == 0) {
      atomicMax(&status[b], (int)TC_ERR_INVALID_ARG);
      best_val[(size_t)b * nB + jb] = -INFINITY;
      best_dst[(size_t)b * nB + jb] = -1;
    }
    return;
  }
  const float inv_b = inv_norm_from_sq(Gb[(size_t)tb * N + tb]);
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  for (int ja = lane; ja < nA; ja += 32) {
    const int ta = setA[(size_t)b * nA + ja];
    if (ta < 0 || ta >= N) {
      atomicMax(&status[b], (int)TC_ERR_INVALID_ARG);
      continue;
    }
    const float inv_a = inv_norm_from_sq(Gb[(size_t)ta * N + ta]);
    const float c = Gb[(size_t)tb * N + ta] * inv_b * inv_a;
    if (c > bv || (c == bv && ta < bi)) {
      bv = c;
      bi = ta;
    }
  }
  warp_best(bv, bi);
  if (lane == 0) {
    best_val[(size_t)b * nB + jb] = bv;
    best_dst[(size_t)b * nB + jb] = (bi == 0x7fffffff) ? -1 : bi;
  }
}

void launch_match_gram(const Dims& D, const float* G, const int32_t* setA, const int32_t* setB,
                       float* best_val, int32_t* best_dst, int32_t* status, cudaStream_t st) {
  Scope scope_(KC_MATCH, st);
  if (D.nB == 0 || D.nA == 0) return;
  dim3 grid((D.nB + 3) / 4, D.B);
  { match_gram_kernel<<<grid, 128, 0, st>>>(G, setA, setB, best_val, best_dst, D.N, D.nA, D.nB, status); note_launch(); }
}

// ------------------------------------------------------------------------------------------
// Eq. 3-10 from the rows of O (stand-alone Stage II): one block per Set-B token keeps its row
// in shared memory as float32; each warp takes Set-A rows in turn.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) match_rows_kernel(const T* __restrict__ O,
                                                        const int32_t* __restrict__ setA,
                                                        const int32_t* __restrict__ setB,
                                                        float* __restrict__ best_val,
                                                        int32_t* __restrict__ best_dst, int N,
                                                        int d, int nA, int nB,
                                                        int32_t* __restrict__ status) {
  extern __shared__ float rowb[];  // [d]
  __shared__ float sv[8];
  __shared__ int si[8];
  __shared__ float s_nb;
  const int b = blockIdx.y, jb = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int tb = setB[(size_t)b * nB + jb];
  const T* Ob = O + (size_t)b * N * d;
  // a token number outside [0, N) in a caller's list is reported and never used as an address
  if (tb < 0 || tb >= N) {
    if (threadIdx.x == 0) {
      atomicMax(&status[b], (int)TC_ERR_INVALID_ARG);
      best_val[(size_t)b * nB + jb] = -INFINITY;
      best_dst[(size_t)b * nB + jb] = -1;
    }
    return;
  }
  for (int c = threadIdx.x; c < d; c += 256) rowb[c] = (float)Ob[(size_t)tb * d + c];
  __syncthreads();
  if (warp == 0) {
    float s = 0.f;
    for (int c = lane; c < d; c += 32) s += rowb[c] * rowb[c];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) s_nb = s;
  }
  __syncthreads();
  const float inv_b = inv_norm_from_sq(s_nb);
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  for (int ja = warp; ja < nA; ja += 8) {
    const int ta = setA[(size_t)b * nA + ja];
    if (ta < 0 || ta >= N) {
      if (lane == 0) atomicMax(&status[b], (int)TC_ERR_INVALID_ARG);
      continue;
    }
    const T* ra = Ob + (size_t)ta * d;
    float dot = 0.f, na = 0.f;
    for (int c = lane; c < d; c += 32) {
      const float v = (float)ra[c];
      dot += v * rowb[c];
      na += v * v;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      dot += __shfl_xor_sync(0xffffffffu, dot, o);
      na += __shfl_xor_sync(0xffffffffu, na, o);
    }
    const float c = dot * inv_b * inv_norm_from_sq(na);
    if (c > bv || (c == bv && ta < bi)) {
      bv = c;
      bi = ta;
    }
  }
  if (lane == 0) {
    sv[warp] = bv;
    si[warp] = bi;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w)
      if (sv[w] > bv || (sv[w] == bv && si[w] < bi)) {
        bv = sv[w];
        bi = si[w];
      }
    best_val[(size_t)b * nB + jb] = bv;
    best_dst[(size_t)b * nB + jb] = (bi == 0x7fffffff) ? -1 : bi;
  }
}

void launch_match_rows(const Dims& D, const void* O, const int32_t* setA, const int32_t* setB,
                       float* best_val, int32_t* best_dst, int32_t* status, cudaStream_t st) {
  Scope scope_(KC_MATCH, st);
  if (D.nB == 0 || D.nA == 0) return;
  dim3 grid(D.nB, D.B);
  size_t smem = (size_t)D.d * sizeof(float);
  TC_WITH_STORAGE_TYPE(D,
    match_rows_kernel<T><<<grid, 256, smem, st>>>((const T*)O, setA, setB, best_val, best_dst, D.N,
                                                  D.d, D.nA, D.nB, status);
    note_launch(););
}

void launch_match_rows_f32(const Dims& D, const float* F, int f, const int32_t* setA,
                           const int32_t* setB, float* best_val, int32_t* best_dst,
                           int32_t* status, cudaStream_t st) {
  Scope scope_(KC_MATCH, st);
  if (D.nB == 0 || D.nA == 0) return;
  dim3 grid(D.nB, D.B);
  { match_rows_kernel<float><<<grid, 256, (size_t)f * sizeof(float), st>>>(F, setA, setB, best_val, best_dst,
                                                                         D.N, f, D.nA, D.nB, status); note_launch(); }
}

// ------------------------------------------------------------------------------------------
// Choice of the M merged Set-B tokens (highest best-similarity, ties to the lower token; Set B
// is in ascending token order so list position is token order), merge lists, kept list.
// One block per image.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(SEL_THREADS) merge_select_kernel(
    const int32_t* __restrict__ setA, const int32_t* __restrict__ setB,
    const float* __restrict__ best_val, const int32_t* __restrict__ best_dst,
    int32_t* __restrict__ msrc, int32_t* __restrict__ mdst, int32_t* __restrict__ kept, int N,
    int nA, int nB, int M, int keep, int32_t* __restrict__ status) {
  extern __shared__ uint32_t dyn[];  // keys [nB] then flags [N] (one word per token)
  uint32_t* keys = dyn;
  uint32_t* flag = dyn + nB;
  __shared__ int hist[256];
  __shared__ uint32_t sh_u[2];
  __shared__ int sh_scan[9];
  const int b = blockIdx.x;
  // Token numbers come from the caller's lists: one outside [0, N) is reported in the image's
  // status and never used as an address (the kept list then ends in -1 entries).
  auto valid = [&](int t) {
    if (t >= 0 && t < N) return true;
    atomicMax(&status[b], (int)TC_ERR_INVALID_ARG);
    return false;
  };
  for (int i = threadIdx.x; i < N; i += SEL_THREADS) flag[i] = 0;
  for (int j = threadIdx.x; j < keep; j += SEL_THREADS) kept[(size_t)b * keep + j] = -1;
  for (int j = threadIdx.x; j < nB; j += SEL_THREADS)
    keys[j] = (M > 0) ? orderable(best_val[(size_t)b * nB + j]) : 0u;
  __syncthreads();
  for (int j = threadIdx.x; j < nA; j += SEL_THREADS) {
    const int t = setA[(size_t)b * nA + j];
    if (valid(t)) flag[t] = 1;
  }
  uint32_t thr = 0xffffffffu;
  int need = 0;
  if (M > 0) block_select_kth(keys, nB, M, hist, sh_u, sh_scan, &thr, &need);

  int tot;
  {
    const int chunk = (nB + SEL_THREADS - 1) / SEL_THREADS;
    const int j0 = min(nB, (int)threadIdx.x * chunk), j1 = min(nB, j0 + chunk);
    int eq = 0;
    for (int j = j0; j < j1; ++j) eq += (keys[j] == thr);
    int e = block_excl_scan(eq, sh_scan, &tot);
    int cm = 0;
    uint32_t sel = 0;  // chunk <= 32
    for (int j = j0; j < j1; ++j) {
      bool in = (M > 0) && (keys[j] > thr);
      if (M > 0 && keys[j] == thr) in = (e++ < need);
      if (in) {
        sel |= 1u << (j - j0);
        ++cm;
      } else {
        const int t = setB[(size_t)b * nB + j];
        if (valid(t)) flag[t] = 1;  // unmerged Set-B tokens stay
      }
    }
    int o = block_excl_scan(cm, sh_scan, &tot);
    for (int j = j0; j < j1; ++j)
      if (sel & (1u << (j - j0))) {
        msrc[(size_t)b * M + o] = setB[(size_t)b * nB + j];
        mdst[(size_t)b * M + o] = best_dst[(size_t)b * nB + j];
        ++o;
      }
  }
  __syncthreads();
  {
    const int chunk = (N + SEL_THREADS - 1) / SEL_THREADS;
    const int i0 = min(N, (int)threadIdx.x * chunk), i1 = min(N, i0 + chunk);
    int c = 0;
    for (int i = i0; i < i1; ++i) c += (int)flag[i];
    int o = block_excl_scan(c, sh_scan, &tot);
    for (int i = i0; i < i1; ++i)
      if (flag[i] && o < keep) kept[(size_t)b * keep + o++] = i;
  }
}

void launch_merge_select(const Dims& D, const int32_t* setA, const int32_t* setB,
                         const float* best_val, const int32_t* best_dst, int32_t* msrc,
                         int32_t* mdst, int32_t* kept, int32_t* status, cudaStream_t st) {
  Scope scope_(KC_MSEL, st);
  size_t smem = (size_t)(D.nB + D.N) * sizeof(uint32_t);
  { merge_select_kernel<<<D.B, SEL_THREADS, smem, st>>>(setA, setB, best_val, best_dst, msrc, mdst,
                                                     kept, D.N, D.nA, D.nB, D.M, D.keep, status); note_launch(); }
}

}  // namespace tc
