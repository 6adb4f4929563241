// G = O O^T for float16 or bfloat16 O on the 5th-generation tensor cores (tcgen05), float32
// accumulate.
//
// The SVD of Sec. 3.3.1 is taken through the Gram matrix (O O^T = U Sigma^2 U^T) and the cosine
// similarities of Eq. 3-10 are its normalised entries, so this is the one dense contraction of
// the path.  One CTA produces one 128 x 128 tile of G for one image:
//   - warp 4 (one lane) streams 128 x 64 slices of the two row blocks of O into a ring of
//     shared-memory stages with TMA (128-byte swizzle, out-of-range rows/columns read as zero);
//   - warp 5 (one lane) issues tcgen05.mma (M = N = 128, K = 16, both operands K-major) into one
//     of two 128-column TMEM accumulators and frees each stage with tcgen05.commit;
//   - warps 0-3 read a finished accumulator back with tcgen05.ld, add it to a float32 register
//     tile, and at the end store the tile and, for a tile below the diagonal, its mirror image,
//     so G is symmetric bit for bit.
// The tensor core adds into its accumulator with truncation, and over the 256 MMA steps of
// d = 4096 that bias reaches 2e-5 relative: enough to move the small singular values the rank
// cut-off sits next to by several 1e-3.  So the K loop is cut into chunks of DRAIN_KB * 64
// elements; each chunk starts a fresh accumulator and the chunk sums are added in registers with
// round-to-nearest, while the tensor core already works on the other accumulator.
// Only tiles on or below the diagonal are computed.  Every mbarrier wait is bounded: a wait
// that runs out records an error for the image and the CTA winds down (TMEM is still freed).
#include "tc_internal.cuh"
#include "tcgen05_util.cuh"

namespace tc {

namespace {

using namespace t5;

constexpr int TILE = 128;         // rows of O per operand tile = tile edge of G
constexpr int BK = 64;            // K elements per stage: 64 halves = one 128-byte swizzle row
constexpr int STAGES = 3;
constexpr int UMMA_K = 16;
constexpr uint32_t TILE_BYTES = TILE * BK * 2;  // 16 KB
constexpr uint32_t SMEM_BYTES = STAGES * 2 * TILE_BYTES + 1024;  // + alignment slack
constexpr uint32_t TMEM_COLS = 256;  // two 128-column accumulators
constexpr int DRAIN_KB = 4;          // stages per accumulation chunk (256 elements of K; 512 breaks the 2e-6 bound)

// Instruction descriptor: D float32, A and B both float16 or both bfloat16 (operand format 0 / 1),
// both K-major, M = 128, N = 128.
constexpr uint32_t IDESC_F16 = (1u << 4) | ((uint32_t)(TILE >> 3) << 17) | ((uint32_t)(TILE >> 4) << 24);
constexpr uint32_t IDESC_BF16 = IDESC_F16 | (1u << 7) | (1u << 10);

__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc,
                                         uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accum)
      : "memory");
}

__global__ void __launch_bounds__(192) gram_tc_kernel(const __grid_constant__ CUtensorMap map,
                                                     float* __restrict__ G, int N, int d,
                                                     int tiles_per_image, int bf16,
                                                     int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[STAGES];
  __shared__ __align__(8) uint64_t bar_empty[STAGES];
  __shared__ __align__(8) uint64_t bar_acc_full[2];
  __shared__ __align__(8) uint64_t bar_acc_empty[2];
  __shared__ uint32_t s_tmem;
  __shared__ int s_fail;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x / tiles_per_image;
  int t = blockIdx.x % tiles_per_image;
  // t -> (ti, tj) with ti >= tj: t = ti (ti + 1) / 2 + tj
  int ti = 0;
  while ((ti + 1) * (ti + 2) / 2 <= t) ++ti;
  const int tj = t - ti * (ti + 1) / 2;
  const bool diag = (ti == tj);
  const int kblocks = (d + BK - 1) / BK;
  const int nchunks = (kblocks + DRAIN_KB - 1) / DRAIN_KB;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  auto stage_a = [&](int s) { return smem_base + (uint32_t)s * 2u * TILE_BYTES; };
  auto stage_b = [&](int s) { return smem_base + (uint32_t)s * 2u * TILE_BYTES + TILE_BYTES; };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bar_acc_full[i]), 1);
      mbar_init(smem_u32(&bar_acc_empty[i]), 4);  // one arrival per epilogue warp
    }
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&s_tmem)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = s_tmem;

  if (warp == 4) {
    // ---- TMA producer ----
    if (lane == 0) {
      for (int kb = 0; kb < kblocks; ++kb) {
        const int s = kb % STAGES;
        const uint32_t round = (uint32_t)(kb / STAGES);
        if (!mbar_wait(smem_u32(&bar_empty[s]), (round & 1u) ^ 1u)) {
          s_fail = 1;
          break;
        }
        const uint32_t full = smem_u32(&bar_full[s]);
        mbar_expect_tx(full, diag ? TILE_BYTES : 2u * TILE_BYTES);
        tma_load_3d(stage_a(s), &map, kb * BK, ti * TILE, b, full);
        if (!diag) tma_load_3d(stage_b(s), &map, kb * BK, tj * TILE, b, full);
      }
    }
  } else if (warp == 5) {
    // ---- MMA issuer ----
    if (lane == 0) {
      bool ok = true;
      for (int c = 0; c < nchunks && ok; ++c) {
        const int buf = c & 1;
        if (!mbar_wait(smem_u32(&bar_acc_empty[buf]), (((uint32_t)c >> 1) & 1u) ^ 1u)) {
          s_fail = 1;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tmem_d = tmem_base + (uint32_t)buf * 128u;
        const int kb_end = min(kblocks, (c + 1) * DRAIN_KB);
        for (int kb = c * DRAIN_KB; kb < kb_end; ++kb) {
          const int s = kb % STAGES;
          const uint32_t round = (uint32_t)(kb / STAGES);
          if (!mbar_wait(smem_u32(&bar_full[s]), round & 1u)) {
            s_fail = 1;
            ok = false;
            break;
          }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t da = umma_desc(stage_a(s));
          const uint64_t db = diag ? da : umma_desc(stage_b(s));
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // 16 halves = 32 bytes further along K inside the swizzled row: +2 in 16-byte units
            umma_f16(tmem_d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), bf16 ? IDESC_BF16 : IDESC_F16,
                     (kb > c * DRAIN_KB || k > 0) ? 1u : 0u);
          }
          umma_commit(smem_u32(&bar_empty[s]));
        }
        umma_commit(smem_u32(&bar_acc_full[buf]));
      }
    }
  } else {
    // ---- epilogue: warps 0..3 own TMEM lanes 32 w .. 32 w + 31 (= rows of the tile) ----
    float acc[TILE];
#pragma unroll
    for (int j = 0; j < TILE; ++j) acc[j] = 0.f;
    bool ok = true;
    for (int c = 0; c < nchunks; ++c) {
      const int buf = c & 1;
      if (!mbar_wait(smem_u32(&bar_acc_full[buf]), ((uint32_t)c >> 1) & 1u)) {
        ok = false;
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)buf * 128u;
#pragma unroll
      for (int q = 0; q < TILE / 32; ++q) {
        float v[32];
        tmem_ld32(taddr + (uint32_t)(q * 32), v);
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[q * 32 + j] += v[j];
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0)
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar_acc_empty[buf]))
                     : "memory");
    }
    // The tile leaves row-major through shared memory (the operand ring is free: every MMA has
    // completed): a thread owns a row, so stores from its registers would put each lane of a
    // store into a sector of its own; from the staging tile a warp writes a whole row per store.
    // The mirror image goes out from the registers (there the lanes are neighbours).
    // All four warps come to the barrier whatever their waits returned.
    constexpr int SROW = TILE + 4;   // floats per staged row
    float* stg = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)));
    if (!ok) s_fail = 1;
    {
      float* srow = stg + (warp * 32 + lane) * SROW;
#pragma unroll
      for (int j = 0; j < TILE / 4; ++j)
        *reinterpret_cast<float4*>(srow + 4 * j) =
            make_float4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (s_fail == 0) {
      float* Gb = G + (size_t)b * N * N;
      for (int rl = warp; rl < TILE; rl += 4) {
        const int grow = ti * TILE + rl;
        if (grow >= N) break;
        const int col = tj * TILE + 4 * lane;
        const float4 v = *reinterpret_cast<const float4*>(stg + rl * SROW + 4 * lane);
        float* dst = Gb + (size_t)grow * N + col;
        if (col + 3 < N && (N & 3) == 0) {
          *reinterpret_cast<float4*>(dst) = v;
        } else {
          if (col < N) dst[0] = v.x;
          if (col + 1 < N) dst[1] = v.y;
          if (col + 2 < N) dst[2] = v.z;
          if (col + 3 < N) dst[3] = v.w;
        }
      }
      const int row = ti * TILE + warp * 32 + lane;
      if (row < N && !diag) {
#pragma unroll
        for (int q = 0; q < TILE / 32; ++q) {
          const int col0 = tj * TILE + q * 32;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (col0 + j < N) Gb[(size_t)(col0 + j) * N + row] = acc[q * 32 + j];
        }
      }
    } else if (status != nullptr) {
      if (threadIdx.x == 0) atomicMax(&status[b], (int)TC_ERR_CUDA);
    } else {
      // no status word to report to: the tile is marked with NaN instead of being left unwritten
      const int row = ti * TILE + warp * 32 + lane;
      if (row < N)
        for (int j = 0; j < TILE; ++j)
          if (tj * TILE + j < N) G[((size_t)b * N + row) * N + tj * TILE + j] = __int_as_float(0x7fc00000);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 5) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(TMEM_COLS)
                 : "memory");
  }
}

}  // namespace

// Returns TC_ERR_UNSUPPORTED when the tensor map cannot be built (caller may not fall back
// silently: it reports the error).
tc_status launch_gram_tc(const Dims& D, const void* O, float* G, int32_t* status, cudaStream_t st) {
  encode_fn enc = get_encode();
  if (enc == nullptr) return TC_ERR_CUDA;
  CUtensorMap map;
  const cuuint64_t dims[3] = {(cuuint64_t)D.d, (cuuint64_t)D.N, (cuuint64_t)D.B};
  const cuuint64_t strides[2] = {(cuuint64_t)D.d * 2, (cuuint64_t)D.N * D.d * 2};
  const cuuint32_t box[3] = {BK, TILE, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(&map, D.bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3,
                   const_cast<void*>(O), dims, strides, box,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return TC_ERR_CUDA;
  if (cudaFuncSetAttribute((const void*)gram_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)SMEM_BYTES) != cudaSuccess)
    return TC_ERR_CUDA;
  const int nt = (D.N + TILE - 1) / TILE;
  const int tiles = nt * (nt + 1) / 2;
  Scope scope_(KC_GRAM, st);
  gram_tc_kernel<<<D.B * tiles, 192, SMEM_BYTES, st>>>(map, G, D.N, D.d, tiles, D.bf16 ? 1 : 0, status);
  note_launch();
  return TC_OK;
}

}  // namespace tc
