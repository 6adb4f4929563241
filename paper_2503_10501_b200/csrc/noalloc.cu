// tc_attn_score_noalloc: Eq. 3-7 for callers that cannot hand the library a workspace.
//
// The attention column-mean runs in two steps: per-chunk partial column sums, then their sum.
// The partial sums need scratch memory.  Every other entry point takes it from the caller's
// workspace; this one takes it from a fixed array that is part of the library image, so the
// caller needs no allocator at all.
#include <mutex>

#include "tc_internal.cuh"

namespace tc {

constexpr size_t kScratchFloats = TC_NOALLOC_SCRATCH_BYTES / sizeof(float);

// Lives in the global memory of every GPU that loads the library, until the process exits.
static __device__ __align__(256) float g_attn_scratch[kScratchFloats];

// In host code `g_attn_scratch` is only a handle for the runtime, not an address the GPU can
// use: the device address has to be asked for, once per device, with that device current.
constexpr int kMaxDevices = 64;
static std::mutex g_mu;
static float* g_scratch_ptr[kMaxDevices] = {nullptr};

static tc_status scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TC_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_mu);
  if (g_scratch_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_attn_scratch) != cudaSuccess || ptr == nullptr) {
      (void)cudaGetLastError();
      return TC_ERR_CUDA;
    }
    g_scratch_ptr[dev] = (float*)ptr;
  }
  *out = g_scratch_ptr[dev];
  return TC_OK;
}

// S[b][x] = (sum over chunks of part[b][c][x]) / (H T), chunks added in index order.
__global__ void __launch_bounds__(256) attn_finish_kernel(const float* __restrict__ part,
                                                         float* __restrict__ S, int N, int chunks,
                                                         float inv_rows) {
  const int b = blockIdx.y;
  const int x = blockIdx.x * 256 + threadIdx.x;
  if (x >= N) return;
  const float* pb = part + (size_t)b * chunks * N;
  float s = 0.f;
  for (int c = 0; c < chunks; ++c) s += pb[(size_t)c * N + x];
  S[(size_t)b * N + x] = s * inv_rows;
}

}  // namespace tc

using namespace tc;

extern "C" tc_status tc_attn_score_noalloc(const tc_params* p, const void* A, float* S,
                                           void* stream) {
  Dims D;
  tc_status s = make_dims(p, &D);
  if (s != TC_OK) return s;
  if (A == nullptr || S == nullptr || ((uintptr_t)A & 15u) != 0) return TC_ERR_INVALID_ARG;
  // this entry point keeps its own, smaller chunk count: its scratch is fixed in size
  {
    const int R = D.H * D.T;
    int chunks = (4 * 148 + D.B - 1) / D.B;
    if (chunks > R / 32) chunks = R / 32;
    if (chunks > 64) chunks = 64;
    if (chunks < 1) chunks = 1;
    D.chunks = chunks;
  }
  const size_t need = (size_t)D.B * D.chunks * D.N;
  if (need > kScratchFloats) return TC_ERR_SCRATCH_LIMIT;
  float* scratch = nullptr;
  s = scratch_for_current_device(&scratch);
  if (s != TC_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  // Every element of the part of the array this call uses is written by the first kernel before
  // the second reads it, so nothing left over from an earlier call has to be cleared.
  launch_attn_colsum(D, A, scratch, st);
  {
    Scope scope_(KC_COMBINE, st);
    dim3 grid((D.N + 255) / 256, D.B);
    attn_finish_kernel<<<grid, 256, 0, st>>>(scratch, S, D.N, D.chunks, 1.0f / (float)(D.H * D.T));
    note_launch();
  }
  return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}
