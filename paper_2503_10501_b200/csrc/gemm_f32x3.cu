// Batched float32-accurate products  C = A B^T  on the 5th-generation tensor cores (tcgen05,
// kind::tf32): the dense products of the subspace solve behind Eq. 3-5 / 3-6 (Sec. 3.3.1).
//
// A float32 value x is used as two TF32 numbers, x ~ hi + lo (both rounded to nearest, so the
// pair is good to 2^-22 |x| and unbiased), and a product as the three tensor-core products
// hi hi + hi lo + lo hi, accumulated in float32.  The operands are plain float32 in memory,
// the contraction index K contiguous in both (A [M][K], B [NN][K]); they are split on the way
// through shared memory.
//
// One CTA produces a 128 x NN tile of C for one image (NN = the whole width of C, a multiple of
// 16; 128, 144, 160 and 192 are built).  Four roles run side by side:
//   - warp 12 (one lane) streams 32-wide K slabs of A and B into a ring of shared-memory stages
//     with TMA (128-byte swizzle, out-of-range rows / K read as zero);
//   - warps 8-11 turn a landed slab into its two parts: hi overwrites the value where it lies,
//     lo goes to the same offset of the stage's second half (the swizzled layout is kept as it
//     is, so nobody has to know it), then a proxy fence hands both to the tensor core;
//   - warp 13 (one lane) issues the twelve tcgen05.mma (M = 128, N = NN, K = 8) of the slab into
//     one of two TMEM accumulators, the small cross terms first, and frees the stage with
//     tcgen05.commit;
//   - warps 0-7 read a finished accumulator back with tcgen05.ld and add it to a float32
//     register tile: the tensor core adds into its accumulator with truncation, so a fresh
//     accumulator every DRAIN_SLABS slabs and round-to-nearest adds in registers keep the bias
//     out.
// The epilogue writes C row-major and / or transposed, as the consumer needs (the consumer wants
// K contiguous again).  Every mbarrier wait is bounded; a wait that runs out records an error for
// the image and the CTA winds down (TMEM is still freed).
#include "tc_internal.cuh"
#include "tcgen05_util.cuh"

namespace tc {

namespace {

using namespace t5;

constexpr int BM = 128;   // rows of C per CTA
constexpr int BK = 32;    // floats of K per stage = one 128-byte swizzle row
constexpr int UK = 8;     // K of one tcgen05.mma kind::tf32
constexpr int EPI_WARPS = 8;     // warps 0-7: accumulator drain and epilogue
constexpr int CONV_WARPS = 4;    // warps 8-11: split of the landed slabs
constexpr int W_TMA = EPI_WARPS + CONV_WARPS, W_MMA = W_TMA + 1;
constexpr int THREADS = (W_MMA + 1) * 32;
constexpr int DRAIN_SLABS = 2;   // slabs accumulated in TMEM before the sum moves to registers
constexpr uint32_t TMEM_COLS = 512;   // two accumulators of up to 256 columns
constexpr uint32_t ACC_STRIDE = 256;

// a stage holds the A slab (128 rows) and the B slab (NN rows), 128 bytes per row, twice:
// values / hi parts in its first half, lo parts in its second
__host__ __device__ constexpr uint32_t a_bytes() { return BM * BK * 4; }
__host__ __device__ constexpr uint32_t half_bytes(int nn) { return a_bytes() + (uint32_t)nn * BK * 4; }
__host__ __device__ constexpr uint32_t stage_bytes(int nn) { return 2 * half_bytes(nn); }
__host__ __device__ constexpr int stages_for(int nn) {
  return (int)((225u * 1024u) / stage_bytes(nn)) > 4 ? 4 : (int)((225u * 1024u) / stage_bytes(nn));
}

__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc,
                                          uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accum)
      : "memory");
}

struct Out {
  float* plain;    // [batch][M][NN]
  float* plainT;   // [batch][NN][M]
};

// NN: width of C (compile time: it sizes the register tile).
template <int NN>
__global__ void __launch_bounds__(THREADS) gemm_f32x3_kernel(const __grid_constant__ CUtensorMap mapA,
                                                           const __grid_constant__ CUtensorMap mapB,
                                                           Out out, int M, int K, int m_tiles,
                                                           int32_t* __restrict__ status) {
  constexpr int STAGES = stages_for(NN);
  constexpr int NCHUNK = NN / 16;            // 16-column chunks of the accumulator
  constexpr int NCH = (NCHUNK + 1) / 2;      // chunks per thread (two column halves)
  constexpr uint32_t A_B = a_bytes(), HALF = half_bytes(NN), STG = stage_bytes(NN);
  // D float32, A and B TF32, both K-major, M = 128, N = NN
  constexpr uint32_t IDESC = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(NN >> 3) << 17) |
                             ((uint32_t)(BM >> 4) << 24);
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[STAGES];    // TMA landed
  __shared__ __align__(8) uint64_t bar_split[STAGES];   // hi / lo of the slab are in place
  __shared__ __align__(8) uint64_t bar_empty[STAGES];   // the MMAs that read the stage are done
  __shared__ __align__(8) uint64_t bar_acc_full[2];
  __shared__ __align__(8) uint64_t bar_acc_empty[2];
  __shared__ uint32_t s_tmem;
  __shared__ int s_fail;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x / m_tiles, mt = blockIdx.x % m_tiles;
  const int slabs = (K + BK - 1) / BK;
  const int nchunks = (slabs + DRAIN_SLABS - 1) / DRAIN_SLABS;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));   // the same place, generic
  auto st_hi = [&](int s) { return smem_base + (uint32_t)s * STG; };
  auto st_lo = [&](int s) { return smem_base + (uint32_t)s * STG + HALF; };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_split[s]), CONV_WARPS);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bar_acc_full[i]), 1);
      mbar_init(smem_u32(&bar_acc_empty[i]), EPI_WARPS);
    }
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == W_MMA) {
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

  if (warp == W_TMA) {
    // ---- TMA producer ----
    if (lane == 0) {
      for (int kb = 0; kb < slabs; ++kb) {
        const int s = kb % STAGES;
        const uint32_t round = (uint32_t)(kb / STAGES);
        if (!mbar_wait(smem_u32(&bar_empty[s]), (round & 1u) ^ 1u)) {
          s_fail = 1;
          break;
        }
        const uint32_t full = smem_u32(&bar_full[s]);
        mbar_expect_tx(full, HALF);
        tma_load_3d(st_hi(s), &mapA, kb * BK, mt * BM, b, full);
        tma_load_3d(st_hi(s) + A_B, &mapB, kb * BK, 0, b, full);
      }
    }
  } else if (warp == W_MMA) {
    // ---- MMA issuer ----
    if (lane == 0) {
      for (int kb = 0; kb < slabs; ++kb) {
        const int c = kb / DRAIN_SLABS, buf = c & 1;
        const bool first = (kb % DRAIN_SLABS) == 0;
        if (first && !mbar_wait(smem_u32(&bar_acc_empty[buf]), (((uint32_t)c >> 1) & 1u) ^ 1u)) {
          s_fail = 1;
          break;
        }
        const int s = kb % STAGES;
        if (!mbar_wait(smem_u32(&bar_split[s]), (uint32_t)(kb / STAGES) & 1u)) {
          s_fail = 1;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tmem_d = tmem_base + (uint32_t)buf * ACC_STRIDE;
        const uint64_t ah = umma_desc(st_hi(s)), al = umma_desc(st_lo(s));
        const uint64_t bh = umma_desc(st_hi(s) + A_B), bl = umma_desc(st_lo(s) + A_B);
        // 8 floats = 32 bytes further along K inside the swizzled row: +2 in 16-byte units.
        // The cross terms go first: what the accumulator truncates while they are added is
        // relative to their own small size.
#pragma unroll
        for (int k = 0; k < BK / UK; ++k)
          umma_tf32(tmem_d, al + (uint64_t)(2 * k), bh + (uint64_t)(2 * k), IDESC, (first && k == 0) ? 0u : 1u);
#pragma unroll
        for (int k = 0; k < BK / UK; ++k)
          umma_tf32(tmem_d, ah + (uint64_t)(2 * k), bl + (uint64_t)(2 * k), IDESC, 1u);
#pragma unroll
        for (int k = 0; k < BK / UK; ++k)
          umma_tf32(tmem_d, ah + (uint64_t)(2 * k), bh + (uint64_t)(2 * k), IDESC, 1u);
        umma_commit(smem_u32(&bar_empty[s]));
        if ((kb % DRAIN_SLABS) == DRAIN_SLABS - 1 || kb == slabs - 1)
          umma_commit(smem_u32(&bar_acc_full[buf]));
      }
    }
  } else if (warp >= EPI_WARPS) {
    // ---- warps 8-11: split every landed slab where it lies ----
    const int t = threadIdx.x - EPI_WARPS * 32;  // 0 .. 127
    constexpr int NV = (int)(HALF / 16);         // float4 per slab
    constexpr int PER = (NV + CONV_WARPS * 32 - 1) / (CONV_WARPS * 32);
    // round to nearest on the bit pattern (ties away from zero, like cvt.rna.tf32): the
    // conversion instruction itself runs at a fraction of the integer rate
    auto rn = [](float x) { return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u); };
    for (int kb = 0; kb < slabs; ++kb) {
      const int s = kb % STAGES;
      if (!mbar_wait(smem_u32(&bar_full[s]), (uint32_t)(kb / STAGES) & 1u)) break;
      float4* hi4 = reinterpret_cast<float4*>(smem_gen + (size_t)s * STG);
      float4* lo4 = reinterpret_cast<float4*>(smem_gen + (size_t)s * STG + HALF);
      constexpr int H1 = (PER + 1) / 2;
#pragma unroll
      for (int part = 0; part < 2; ++part) {   // two batches, the loads of a batch in flight together
        const int j0 = part ? H1 : 0, j1 = part ? PER : H1;
        float4 x[H1];
#pragma unroll
        for (int j = j0; j < j1; ++j) {
          const int i = t + j * CONV_WARPS * 32;
          if (i < NV) x[j - j0] = hi4[i];
        }
#pragma unroll
        for (int j = j0; j < j1; ++j) {
          const int i = t + j * CONV_WARPS * 32;
          if (i < NV) {
            const float4 v = x[j - j0];
            float4 h, l;
            h.x = rn(v.x); l.x = rn(v.x - h.x);
            h.y = rn(v.y); l.y = rn(v.y - h.y);
            h.z = rn(v.z); l.z = rn(v.z - h.z);
            h.w = rn(v.w); l.w = rn(v.w - h.w);
            hi4[i] = h;
            lo4[i] = l;
          }
        }
      }
      // make the generic-proxy writes visible to the tensor core's reads of shared memory
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0)
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar_split[s])) : "memory");
    }
  } else {
    // ---- warps 0-7: drain the accumulators, then the epilogue.  Warp w owns TMEM lanes
    //      32 (w % 4) .. + 31 (rows of the tile) and the 16-column chunks half, half + 2, ...
    //      with half = w / 4 ----
    const int quad = warp & 3, half = warp >> 2;
    float acc[NCH][16];
#pragma unroll
    for (int c = 0; c < NCH; ++c)
#pragma unroll
      for (int j = 0; j < 16; ++j) acc[c][j] = 0.f;
    bool ok = true;
    for (int ch = 0; ch < nchunks; ++ch) {
      const int buf = ch & 1;
      if (!mbar_wait(smem_u32(&bar_acc_full[buf]), ((uint32_t)ch >> 1) & 1u)) {
        ok = false;
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)buf * ACC_STRIDE;
      // two loads in flight at a time
#pragma unroll
      for (int c = 0; c < NCH; c += 2) {
        uint32_t v[2][16];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int chunk = 2 * (c + u) + half;
          if (c + u < NCH && chunk < NCHUNK) tmem_ld16_issue(taddr + (uint32_t)(chunk * 16), v[u]);
        }
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int chunk = 2 * (c + u) + half;
          if (c + u < NCH && chunk < NCHUNK) {
#pragma unroll
            for (int j = 0; j < 16; ++j) acc[c + u][j] += __uint_as_float(v[u][j]);
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0)
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar_acc_empty[buf]))
                     : "memory");
    }
    // The row-major form leaves through shared memory (the operand ring is free: every MMA that
    // read it has completed): a thread owns a row of the tile, so stores straight from its
    // registers would put every lane into a sector of its own; from the staging tile a warp
    // writes whole rows.  All eight warps come to the barrier whatever their waits returned.
    constexpr int SROW = NN + 4;   // floats per staged row: 16-byte aligned, no bank hit twice by a quarter warp
    float* stg = reinterpret_cast<float*>(smem_gen);
    if (!ok) s_fail = 1;
    if (out.plain != nullptr) {
      float* srow = stg + (quad * 32 + lane) * SROW;
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const int chunk = 2 * c + half;
        if (chunk >= NCHUNK) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          *reinterpret_cast<float4*>(srow + chunk * 16 + 4 * j) =
              make_float4(acc[c][4 * j], acc[c][4 * j + 1], acc[c][4 * j + 2], acc[c][4 * j + 3]);
      }
    }
    asm volatile("bar.sync 2, 256;" ::: "memory");
    if (s_fail == 0) {
      const size_t MN = (size_t)M * NN;
      if (out.plain != nullptr) {
        for (int rl = warp; rl < BM; rl += EPI_WARPS) {
          const int grow = mt * BM + rl;
          if (grow >= M) break;
          const float4* src = reinterpret_cast<const float4*>(stg + rl * SROW);
          float4* dst = reinterpret_cast<float4*>(out.plain + (size_t)b * MN + (size_t)grow * NN);
          for (int v = lane; v < NN / 4; v += 32) dst[v] = src[v];
        }
      }
      const int row = mt * BM + quad * 32 + lane;
      if (row < M && out.plainT != nullptr) {
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          const int chunk = 2 * c + half;
          if (chunk >= NCHUNK) continue;
          float* dst = out.plainT + (size_t)b * MN + (size_t)(chunk * 16) * M + row;
#pragma unroll
          for (int j = 0; j < 16; ++j) dst[(size_t)j * M] = acc[c][j];
        }
      }
    } else if (status != nullptr && threadIdx.x == 0) {
      atomicMax(&status[b], (int)TC_ERR_CUDA);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == W_MMA) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(TMEM_COLS)
                 : "memory");
  }
}

// [K, rows, batch] float32, box 32 x box_rows x 1, 128-byte swizzle, zero fill
bool encode_operand(CUtensorMap* map, const float* base, int rows, int K, int batch, int box_rows) {
  encode_fn enc = get_encode();
  if (enc == nullptr) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)batch};
  const cuuint64_t strides[2] = {(cuuint64_t)K * 4, (cuuint64_t)rows * K * 4};
  const cuuint32_t box[3] = {BK, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int NN>
tc_status launch_nn(const CUtensorMap& mapA, const CUtensorMap& mapB, const Out& out, int M, int K,
                    int batch, int32_t* status, cudaStream_t st) {
  constexpr uint32_t smem = (uint32_t)stages_for(NN) * stage_bytes(NN) + 1024;
  if (cudaFuncSetAttribute((const void*)gemm_f32x3_kernel<NN>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return TC_ERR_CUDA;
  const int m_tiles = (M + BM - 1) / BM;
  gemm_f32x3_kernel<NN><<<batch * m_tiles, THREADS, smem, st>>>(mapA, mapB, out, M, K, m_tiles, status);
  note_launch();
  return TC_OK;
}

}  // namespace

bool gemm_f32x3_supported(int M, int NN, int K) {
  if (M < 1 || K < 4 || (K & 3) != 0) return false;  // TMA rows are whole 16-byte vectors
  return NN == 128 || NN == 144 || NN == 160 || NN == 192;
}

// C [batch][M][NN] = A B^T with A [batch][M][K], B [batch][NN][K] float32, 16-byte aligned.
tc_status launch_gemm_f32x3(const float* A, const float* B, int M, int NN, int K, int batch,
                            float* C, float* CT, int32_t* status, cudaStream_t st, int cls) {
  if (!gemm_f32x3_supported(M, NN, K)) return TC_ERR_UNSUPPORTED;
  CUtensorMap mapA, mapB;
  if (!encode_operand(&mapA, A, M, K, batch, BM) || !encode_operand(&mapB, B, NN, K, batch, NN))
    return TC_ERR_CUDA;
  Out out{C, CT};
  Scope scope_(cls, st);
  switch (NN) {
    case 128: return launch_nn<128>(mapA, mapB, out, M, K, batch, status, st);
    case 144: return launch_nn<144>(mapA, mapB, out, M, K, batch, status, st);
    case 160: return launch_nn<160>(mapA, mapB, out, M, K, batch, status, st);
    case 192: return launch_nn<192>(mapA, mapB, out, M, K, batch, status, st);
    default: return TC_ERR_UNSUPPORTED;
  }
}

}  // namespace tc
