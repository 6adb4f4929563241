// HBM-streaming kernels of the carve path: attention column sums (Eq. 3-7), score combination
// (Eq. 3-8) and the merge + gather of X, K, V (Sec. 3.3.2, last paragraph).
#include "tc_internal.cuh"

namespace tc {

// ------------------------------------------------------------------------------------------
// 16-byte vector helpers: a vector holds 8 halves or 4 floats.
// ------------------------------------------------------------------------------------------
template <typename T>
struct Vec16;
template <>
struct Vec16<__half> {
  static constexpr int L = 8;
  __device__ static void unpack(const uint4& v, float* f) {
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 t = __half22float2(h[i]);
      f[2 * i] = t.x;
      f[2 * i + 1] = t.y;
    }
  }
  __device__ static uint4 pack(const float* f) {
    uint4 v;
    __half2* h = reinterpret_cast<__half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2half2_rn(f[2 * i], f[2 * i + 1]);
    return v;
  }
};
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int L = 8;
  __device__ static void unpack(const uint4& v, float* f) {
    // a bfloat16 is the upper half of a float32
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static uint4 pack(const float* f) {
    uint4 v;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    return v;
  }
};
template <>
struct Vec16<float> {
  static constexpr int L = 4;
  __device__ static void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x);
    f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z);
    f[3] = __uint_as_float(v.w);
  }
  __device__ static uint4 pack(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                      __float_as_uint(f[3]));
  }
};

__device__ inline float to_f32(__half v) { return __half2float(v); }
__device__ inline float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ inline float to_f32(float v) { return v; }

// ------------------------------------------------------------------------------------------
// Eq. 3-7, first half: per image and per chunk of the H*T attention rows, the column sums.
// grid (chunks, B); block (bx, by): x walks 16-byte column groups, y walks rows.
// part[b][chunk][x] is written by exactly one block, in a fixed summation order.
// ------------------------------------------------------------------------------------------
template <typename T, bool VECTOR>
__global__ void attn_colsum_kernel(const T* __restrict__ A, float* __restrict__ part, int R,
                                   int N, int rows_per_chunk) {
  constexpr int L = VECTOR ? Vec16<T>::L : 1;
  extern __shared__ float red[];  // [by][bx * L]
  const int b = blockIdx.y, chunk = blockIdx.x;
  const int bx = blockDim.x, by = blockDim.y;
  const int ncg = N / L;
  const int r_begin = chunk * rows_per_chunk;
  const int r_end = min(R, r_begin + rows_per_chunk);
  const T* Ab = A + (size_t)b * R * N;
  float* out = part + ((size_t)b * gridDim.x + chunk) * N;

  for (int cg0 = 0; cg0 < ncg; cg0 += bx) {
    const int cg = cg0 + threadIdx.x;
    float acc[L];
#pragma unroll
    for (int i = 0; i < L; ++i) acc[i] = 0.f;
    if (cg < ncg) {
      int r = r_begin + threadIdx.y;
      if (VECTOR) {
        // eight independent 16-byte loads in flight per thread
        for (; r + 7 * by < r_end; r += 8 * by) {
          uint4 v[8];
#pragma unroll
          for (int u = 0; u < 8; ++u)
            v[u] = __ldg(reinterpret_cast<const uint4*>(Ab + (size_t)(r + u * by) * N) + cg);
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            float f[8];
            Vec16<T>::unpack(v[u], f);
#pragma unroll
            for (int i = 0; i < L; ++i) acc[i] += f[i];
          }
        }
        for (; r < r_end; r += by) {
          uint4 v = __ldg(reinterpret_cast<const uint4*>(Ab + (size_t)r * N) + cg);
          float f[8];
          Vec16<T>::unpack(v, f);
#pragma unroll
          for (int i = 0; i < L; ++i) acc[i] += f[i];
        }
      } else {
        for (; r < r_end; r += by) acc[0] += to_f32(Ab[(size_t)r * N + cg]);
      }
    }
#pragma unroll
    for (int i = 0; i < L; ++i) red[(threadIdx.y * bx + threadIdx.x) * L + i] = acc[i];
    __syncthreads();
    if (threadIdx.y == 0 && cg < ncg) {
#pragma unroll
      for (int i = 0; i < L; ++i) {
        float s = 0.f;
        for (int y = 0; y < by; ++y) s += red[(y * bx + threadIdx.x) * L + i];
        out[cg * L + i] = s;
      }
    }
    __syncthreads();
  }
}

void launch_attn_colsum(const Dims& D, const void* A, float* s_part, cudaStream_t st) {
  Scope scope_(KC_ATTN, st);
  const int R = D.H * D.T;
  const int L = 16 / D.esz;
  const bool vec = (D.N % L) == 0;
  const int ncg = vec ? D.N / L : D.N;
  int bx = min(ncg, 128);
  bx = (bx + 31) / 32 * 32;
  int by = max(1, 256 / bx);
  const int rpc = (R + D.chunks - 1) / D.chunks;
  dim3 grid(D.chunks, D.B), block(bx, by);
  size_t smem = (size_t)bx * by * (vec ? L : 1) * sizeof(float);
  TC_WITH_STORAGE_TYPE(D,
    if (vec) { attn_colsum_kernel<T, true><<<grid, block, smem, st>>>((const T*)A, s_part, R, D.N, rpc); }
    else { attn_colsum_kernel<T, false><<<grid, block, smem, st>>>((const T*)A, s_part, R, D.N, rpc); }
    note_launch(););
}

// ------------------------------------------------------------------------------------------
// Eq. 3-7 second half and Eq. 3-8: S = colsum / (H T);  E = (1 - lambda) C~ + lambda S~.
// One block per image; all reductions run in a fixed order.
// ------------------------------------------------------------------------------------------
__device__ float block_sum_256(float v, float* sh) {
  const int t = threadIdx.x;
  sh[t] = v;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (t < s) sh[t] += sh[t + s];
    __syncthreads();
  }
  float r = sh[0];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(256) combine_kernel(const float* __restrict__ part,
                                                     const float* __restrict__ C,
                                                     float* __restrict__ S, float* __restrict__ E,
                                                     int N, int chunks, float inv_rows,
                                                     float lambda, int sum1) {
  __shared__ float sh[256];
  const int b = blockIdx.x;
  const float* pb = part + (size_t)b * chunks * N;
  float ls = 0.f, lc = 0.f;
  for (int x = threadIdx.x; x < N; x += 256) {
    // chunk partials are added in chunk order, eight loads in flight at a time
    float s = 0.f;
    int c = 0;
    for (; c + 7 < chunks; c += 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = pb[(size_t)(c + u) * N + x];
#pragma unroll
      for (int u = 0; u < 8; ++u) s += v[u];
    }
    for (; c < chunks; ++c) s += pb[(size_t)c * N + x];
    s *= inv_rows;
    S[(size_t)b * N + x] = s;
    ls += s;
    lc += C[(size_t)b * N + x];
  }
  float cs = 1.f, ss = 1.f;
  if (sum1) {
    ss = block_sum_256(ls, sh);
    cs = block_sum_256(lc, sh);
    if (!(ss > 0.f)) ss = 1.f;
    if (!(cs > 0.f)) cs = 1.f;
  }
  __syncthreads();
  for (int x = threadIdx.x; x < N; x += 256) {
    float c = C[(size_t)b * N + x], s = S[(size_t)b * N + x];
    if (sum1) {
      c = c / cs;
      s = s / ss;
    }
    E[(size_t)b * N + x] = (1.f - lambda) * c + lambda * s;
  }
}

void launch_combine(const Dims& D, const float* s_part, const float* C, float* S, float* E,
                    cudaStream_t st) {
  Scope scope_(KC_COMBINE, st);
  const float inv_rows = 1.0f / (float)(D.H * D.T);
  { combine_kernel<<<D.B, 256, 0, st>>>(s_part, C, S, E, D.N, D.chunks, inv_rows, D.lambda,
                                      D.score_norm == TC_NORM_SUM1 ? 1 : 0); note_launch(); }
}

// ------------------------------------------------------------------------------------------
// Merge + gather.  grid (keep, B), block 256.  Block (j, b) produces output row j of image b
// for X and for every head of K and V: the mean of token a = kept[j] and of every token whose
// merge destination is a, or a bit-exact copy when nothing merges into a.
// ------------------------------------------------------------------------------------------
template <typename T>
__device__ inline void merge_row(const T* __restrict__ base, size_t row_stride, int a,
                                 const int* srcs, int cnt, T* __restrict__ out, int nvec,
                                 int v0, int vstep, const float* wts) {
  // wts: null for the plain mean, else wts[0] = weight of a, wts[1 + s] of source s, and
  // wts[cnt + 1] = 1 / their sum
  constexpr int L = Vec16<T>::L;
  const uint4* pa = reinterpret_cast<const uint4*>(base + (size_t)a * row_stride);
  uint4* po = reinterpret_cast<uint4*>(out);
  for (int v = v0; v < nvec; v += vstep) {
    uint4 va = __ldg(pa + v);
    if (cnt == 0) {
      po[v] = va;
      continue;
    }
    float acc[8], f[8];
    Vec16<T>::unpack(va, acc);
    if (wts != nullptr) {
      const float wa = wts[0];
#pragma unroll
      for (int i = 0; i < L; ++i) acc[i] *= wa;
    }
    for (int s = 0; s < cnt; ++s) {
      uint4 vs = __ldg(reinterpret_cast<const uint4*>(base + (size_t)srcs[s] * row_stride) + v);
      Vec16<T>::unpack(vs, f);
      if (wts != nullptr) {
        const float w = wts[1 + s];
#pragma unroll
        for (int i = 0; i < L; ++i) acc[i] = fmaf(w, f[i], acc[i]);
      } else {
#pragma unroll
        for (int i = 0; i < L; ++i) acc[i] += f[i];
      }
    }
    if (wts != nullptr) {
      const float inv = wts[cnt + 1];
#pragma unroll
      for (int i = 0; i < L; ++i) acc[i] *= inv;
    } else {
      const float den = (float)(cnt + 1);
#pragma unroll
      for (int i = 0; i < L; ++i) acc[i] = acc[i] / den;
    }
    po[v] = Vec16<T>::pack(acc);
  }
}

template <typename T>
__global__ void __launch_bounds__(256) compact_kernel(
    const T* __restrict__ X, const T* __restrict__ K, const T* __restrict__ V,
    const int32_t* __restrict__ kept, const int32_t* __restrict__ msrc,
    const int32_t* __restrict__ mdst, T* __restrict__ Xo, T* __restrict__ Ko,
    T* __restrict__ Vo, int N, int d, int H, int dh, int keep, int M,
    const float* __restrict__ E, int32_t* __restrict__ status) {
  extern __shared__ int srcs[];  // [M] sources, then [M + 2] floats of weights
  float* wts_sm = reinterpret_cast<float*>(srcs + M);
  __shared__ int s_cnt;
  __shared__ int s_weighted;
  constexpr int L = Vec16<T>::L;
  const int b = blockIdx.y, j = blockIdx.x;
  const int a = kept[(size_t)b * keep + j];
  // The lists may come from the caller: a token number outside [0, N) is reported in the
  // image's status and never used as an address.  A bad kept entry gives a row of zeros, a bad
  // source is left out of its group.
  if (a < 0 || a >= N) {
    if (threadIdx.x == 0) atomicMax(&status[b], (int)TC_ERR_INVALID_ARG);
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    uint4* xo = reinterpret_cast<uint4*>(Xo + ((size_t)b * keep + j) * d);
    for (int v = threadIdx.x; v < d / L; v += 256) xo[v] = z;
    if (K != nullptr) {
      const int vpr = dh / L;
      for (int idx = threadIdx.x; idx < H * vpr; idx += 256) {
        const int h = idx / vpr, v = idx - h * vpr;
        const size_t out_off = (((size_t)b * H + h) * keep + j) * dh;
        reinterpret_cast<uint4*>(Ko + out_off)[v] = z;
        reinterpret_cast<uint4*>(Vo + out_off)[v] = z;
      }
    }
    return;
  }
  // ordered list of the sources merged into a (first warp, ballot compaction)
  if (threadIdx.x < 32) {
    int cnt = 0;
    for (int m0 = 0; m0 < M; m0 += 32) {
      const int m = m0 + threadIdx.x;
      bool hit = (m < M) && (mdst[(size_t)b * M + m] == a);
      if (hit) {
        const int sidx = msrc[(size_t)b * M + m];
        if (sidx < 0 || sidx >= N) {
          atomicMax(&status[b], (int)TC_ERR_INVALID_ARG);
          hit = false;
        }
      }
      const unsigned mask = __ballot_sync(0xffffffffu, hit);
      if (hit) srcs[cnt + __popc(mask & ((1u << threadIdx.x) - 1u))] = msrc[(size_t)b * M + m];
      cnt += __popc(mask);
    }
    if (threadIdx.x == 0) {
      s_cnt = cnt;
      // score-weighted variant: the group's weights and the reciprocal of their sum; a sum
      // that is not positive falls back to the plain mean
      int weighted = 0;
      if (E != nullptr && cnt > 0) {
        const float* Eb = E + (size_t)b * N;
        float tot = Eb[a];
        wts_sm[0] = Eb[a];
        for (int q = 0; q < cnt; ++q) {
          wts_sm[1 + q] = Eb[srcs[q]];
          tot += Eb[srcs[q]];
        }
        if (tot > 0.f) {
          wts_sm[cnt + 1] = 1.0f / tot;
          weighted = 1;
        }
      }
      s_weighted = weighted;
    }
  }
  __syncthreads();
  const int cnt = s_cnt;
  const float* wts = s_weighted ? wts_sm : nullptr;

  // X row
  merge_row<T>(X + (size_t)b * N * d, d, a, srcs, cnt, Xo + ((size_t)b * keep + j) * d, d / L,
               threadIdx.x, 256, wts);
  // K, V rows of every head
  if (K != nullptr) {
    const int vpr = dh / L;
    for (int idx = threadIdx.x; idx < H * vpr; idx += 256) {
      const int h = idx / vpr, v = idx - h * vpr;
      const size_t in_off = ((size_t)b * H + h) * N * dh;
      const size_t out_off = (((size_t)b * H + h) * keep + j) * dh;
      merge_row<T>(K + in_off, dh, a, srcs, cnt, Ko + out_off, v + 1, v, vpr + 1, wts);
      merge_row<T>(V + in_off, dh, a, srcs, cnt, Vo + out_off, v + 1, v, vpr + 1, wts);
    }
  }
}

void launch_compact(const Dims& D, const void* X, const void* K, const void* V,
                    const int32_t* kept, const int32_t* msrc, const int32_t* mdst, void* Xo,
                    void* Ko, void* Vo, const float* E, int32_t* status, cudaStream_t st) {
  Scope scope_(KC_COMPACT, st);
  dim3 grid(D.keep, D.B);
  size_t smem = (size_t)max(D.M, 1) * sizeof(int) + (size_t)(D.M + 2) * sizeof(float);
  TC_WITH_STORAGE_TYPE(D,
    compact_kernel<T><<<grid, 256, smem, st>>>((const T*)X, (const T*)K, (const T*)V, kept, msrc, mdst,
                                               (T*)Xo, (T*)Ko, (T*)Vo, D.N, D.d, D.H, D.dh, D.keep,
                                               D.M, E, status);
    note_launch(););
}

// ------------------------------------------------------------------------------------------
// Km[b][x][:] = mean over the heads h of K[b][h][x][:], float32 (the features ToMe matches on).
// grid (N, B), block dh (rounded up to a warp).
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void mean_heads_kernel(const T* __restrict__ K, float* __restrict__ Km, int H, int N,
                                  int dh) {
  const int x = blockIdx.x, b = blockIdx.y;
  const float inv = 1.0f / (float)H;
  for (int c = threadIdx.x; c < dh; c += blockDim.x) {
    float s = 0.f;
    for (int h = 0; h < H; ++h) s += to_f32(K[(((size_t)b * H + h) * N + x) * dh + c]);
    Km[((size_t)b * N + x) * dh + c] = s * inv;
  }
}

void launch_mean_heads(const Dims& D, const void* K, float* Km, cudaStream_t st) {
  Scope scope_(KC_MATCH, st);
  dim3 grid(D.N, D.B);
  const int threads = min(256, (D.dh + 31) / 32 * 32);
  TC_WITH_STORAGE_TYPE(D,
    mean_heads_kernel<T><<<grid, threads, 0, st>>>((const T*)K, Km, D.H, D.N, D.dh);
    note_launch(););
}

// ------------------------------------------------------------------------------------------
// Rows idx[b][0..n_sub) of O [B, N, d] copied to Os [B, n_sub, d] (Sec. 3.2: the rows of the
// attention output that belong to a set of tokens).  grid (n_sub, B); 16-byte vectors.  An
// index outside [0, N) gives a zero row and TC_ERR_INVALID_ARG in the image's status.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) gather_rows_kernel(const uint4* __restrict__ O,
                                                         const int32_t* __restrict__ idx,
                                                         uint4* __restrict__ Os, int N, int n_sub,
                                                         int vec_per_row,
                                                         int32_t* __restrict__ status) {
  const int b = blockIdx.y, j = blockIdx.x;
  const int t = idx[(size_t)b * n_sub + j];
  const bool ok = t >= 0 && t < N;
  if (!ok && threadIdx.x == 0) atomicMax(&status[b], (int)TC_ERR_INVALID_ARG);
  const uint4* src = O + ((size_t)b * N + (ok ? t : 0)) * vec_per_row;
  uint4* dst = Os + ((size_t)b * n_sub + j) * vec_per_row;
  for (int v = threadIdx.x; v < vec_per_row; v += 128)
    dst[v] = ok ? __ldg(src + v) : make_uint4(0u, 0u, 0u, 0u);
}

void launch_gather_rows(const Dims& D, int n_sub, const void* O, const int32_t* idx, void* Os,
                        int32_t* status, cudaStream_t st) {
  Scope scope_(KC_COMPACT, st);
  dim3 grid(n_sub, D.B);
  { gather_rows_kernel<<<grid, 128, 0, st>>>((const uint4*)O, idx, (uint4*)Os, D.N, n_sub,
                                            D.d * D.esz / 16, status); note_launch(); }
}

// ------------------------------------------------------------------------------------------
// Sequence after the compression (Sec. 3.1: [system, visual, prompt]; Conclusion: original
// position IDs are kept).  Output row j of image b: a system row, compacted visual row
// j - n_sys, or a prompt row, with its original position.  grid (L_out, B); 16-byte vectors.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) reassemble_kernel(const uint4* __restrict__ Hs,
                                                        const uint4* __restrict__ Xo,
                                                        const int32_t* __restrict__ kept,
                                                        uint4* __restrict__ Ho,
                                                        int32_t* __restrict__ pos, int n_sys,
                                                        int n_vis, int n_text, int keep,
                                                        int vec_per_row) {
  const int b = blockIdx.y, j = blockIdx.x;
  const int L = n_sys + n_vis + n_text, Lo = n_sys + keep + n_text;
  const uint4* src;
  int p;
  if (j < n_sys) {
    p = j;
    src = Hs + ((size_t)b * L + j) * vec_per_row;
  } else if (j < n_sys + keep) {
    p = n_sys + kept[(size_t)b * keep + j - n_sys];
    src = Xo + ((size_t)b * keep + j - n_sys) * vec_per_row;
  } else {
    p = j - keep + n_vis;
    src = Hs + ((size_t)b * L + p) * vec_per_row;
  }
  uint4* dst = Ho + ((size_t)b * Lo + j) * vec_per_row;
  for (int v = threadIdx.x; v < vec_per_row; v += 128) dst[v] = __ldg(src + v);
  if (threadIdx.x == 0) pos[(size_t)b * Lo + j] = p;
}

void launch_reassemble(const Dims& D, int n_sys, int n_text, const void* Hs, const void* Xo,
                       const int32_t* kept, void* Ho, int32_t* pos, cudaStream_t st) {
  Scope scope_(KC_COMPACT, st);
  dim3 grid(n_sys + D.keep + n_text, D.B);
  { reassemble_kernel<<<grid, 128, 0, st>>>((const uint4*)Hs, (const uint4*)Xo, kept, (uint4*)Ho, pos,
                                           n_sys, D.N, n_text, D.keep, D.d * D.esz / 16); note_launch(); }
}

// ------------------------------------------------------------------------------------------
// Rotary-encoding tables for rows with given position IDs (Conclusion: the later layers rotate
// by the original positions): cos / sin of pos * base^(-2 i / dh), i < dh / 2.  The angle is
// formed and reduced in double precision (a float32 angle of a few thousand radians would cost
// four digits); the tables are float32.  grid = rows, block = dh / 2 rounded up to a warp.
// ------------------------------------------------------------------------------------------
__global__ void rope_tables_kernel(const int32_t* __restrict__ pos, int half, double neg_log2_base_2_over_dh,
                                   float* __restrict__ cosv, float* __restrict__ sinv) {
  const size_t row = blockIdx.x;
  const double p = (double)pos[row];
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    const double theta = exp2(neg_log2_base_2_over_dh * (double)i);
    double sn, cs;
    sincos(p * theta, &sn, &cs);
    cosv[row * half + i] = (float)cs;
    sinv[row * half + i] = (float)sn;
  }
}

void launch_rope_tables(const int32_t* pos, long long rows, int head_dim, double base, float* cosv,
                        float* sinv, cudaStream_t st) {
  Scope scope_(KC_COMPACT, st);
  const int half = head_dim / 2;
  const int threads = min(256, (half + 31) / 32 * 32);
  { rope_tables_kernel<<<(unsigned)rows, threads, 0, st>>>(pos, half, -2.0 * log2(base) / (double)head_dim,
                                                         cosv, sinv); note_launch(); }
}

}  // namespace tc
