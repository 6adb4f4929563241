// The layer-2 probe: from the queries, keys and values of one attention layer on the sequence
// [system, visual, prompt] (Sec. 3.1), the two things the compression reads: the visual rows of
// Z = Softmax(Q K^T / sqrt(d_k)) V (Eq. 3-1, 3-2; heads side by side), and the attention the
// probe rows pay to the visual tokens (the slice Eq. 3-7 averages).  The probability matrix is
// never written out in full.
//
// Both products run on the 5th-generation tensor cores (tcgen05.mma kind::f16, M = N = 128,
// float32 accumulators in TMEM, operands staged by TMA with the 128-byte swizzle).  One CTA owns
// 128 query rows of one head of one image and walks the keys in blocks of 128:
//   - warp 8 (one lane): TMA loads of the query tile (once), then per block the key tile and,
//     when Z is wanted, the tile of V^T (V is transposed into the workspace first, so that both
//     operands of P V have their contraction index contiguous);
//   - warp 9 (one lane): S = Q K^T into TMEM; later O_blk = P V into a second accumulator;
//   - warps 0-7: two threads per query row, each with half of the block's 128 columns (and half
//     of the row of Z).  The scores come back with tcgen05.ld, get the causal mask, and feed an
//     online softmax in the exp2 domain (the two halves of a row exchange their block maxima
//     through shared memory); the probabilities are written as
//     float16 / bfloat16 into a shared-memory tile of their own (in the swizzled layout the
//     tensor core expects), and the block's P V is folded into a float32 row of Z held in
//     registers, rescaled when the running maximum moves.
// The scores have two accumulators and V^T two tiles: while the softmax warps work on block i the
// tensor core already forms the scores of block i + 1, and the loads of block i + 1 are in flight.
// The probe rows take two passes over the keys instead (first the row maxima and sums, then the
// normalised probabilities of the visual columns) and need no V.
// Every mbarrier wait is bounded; a wait that runs out records an error for the image and the
// CTA winds down (TMEM is still freed).
#include "tc_internal.cuh"
#include "tcgen05_util.cuh"

namespace tc {

namespace {

using namespace t5;

constexpr int QT = 128;          // query rows per CTA
constexpr int KB = 128;          // keys per block
constexpr int DH = 128;          // head dimension the kernel is built for
constexpr uint32_t ATOM = 128 * 128;        // bytes of one 128-row x 64-element swizzle atom
constexpr uint32_t TILE_B = 2 * ATOM;       // a 128 x 128 tile of 16-bit elements
constexpr uint32_t SMEM_O = 6 * TILE_B + 1024;   // Q, K, two tiles of P, two tiles of V^T
constexpr uint32_t STG_ROW = 2 * KB + 16;         // bytes of a row of the staging tile (padded: no bank is hit twice by a quarter warp)
constexpr uint32_t SMEM_A = 2 * TILE_B + QT * STG_ROW + 1024;   // Q, K, staging tile of the probabilities
constexpr uint32_t TMEM_COLS_O = 512;            // two score accumulators and two for the blocks' P V
constexpr uint32_t TMEM_COLS_A = 256;            // two score accumulators

// D float32, A and B float16 (bf = 0) or bfloat16 (bf = 1), both K-major, M = N = 128
__device__ __forceinline__ uint32_t idesc(int bf) {
  return (1u << 4) | (bf ? ((1u << 7) | (1u << 10)) : 0u) | ((uint32_t)(128 >> 3) << 17) |
         ((uint32_t)(128 >> 4) << 24);
}

__device__ __forceinline__ void umma_16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t id,
                                        uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(id), "r"(accum)
      : "memory");
}

// the eight tcgen05.mma of a 128 x 128 x 128 product of two swizzled 16-bit tiles
__device__ __forceinline__ void mma_tile(uint32_t tmem_d, uint32_t a_base, uint32_t b_base, uint32_t id) {
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    const uint32_t atom = (uint32_t)(ks >> 2) * ATOM;
    umma_16(tmem_d, umma_desc(a_base + atom) + (uint64_t)(2 * (ks & 3)),
            umma_desc(b_base + atom) + (uint64_t)(2 * (ks & 3)), id, ks > 0 ? 1u : 0u);
  }
}

__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 2^x on the special-function unit (relative error 2^-22: far inside the 16-bit outputs)
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <typename T>
__device__ __forceinline__ uint32_t pack2(float a, float b);
template <>
__device__ __forceinline__ uint32_t pack2<__half>(float a, float b) {
  __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
template <>
__device__ __forceinline__ uint32_t pack2<__nv_bfloat16>(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

struct ProbeArgs {
  int L, n_sys, n_vis, H;
  int row0;          // sequence position of the first query row this launch covers
  int n_rows;        // number of query rows
  float scale2;      // log2(e) / sqrt(dh)
  int bf;
};

// WANT_O: visual query rows -> rows of Z (O_out [B][n_vis][H * dh]).
// !WANT_O: probe rows -> probabilities of the visual columns (A_out [B][H][n_rows][n_vis]).
template <typename T, bool WANT_O>
__global__ void __launch_bounds__(320, 1) probe_kernel(
    const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
    const __grid_constant__ CUtensorMap mapVt, ProbeArgs pa, T* __restrict__ out,
    int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  // bar_k: key tile landed; bar_kfree: its scores are formed (the tile may be reloaded);
  // bar_v[2]: V^T tile landed; bar_s[2]: scores ready in accumulator 0 / 1; bar_sfree[2]: the
  // softmax warps are done with that accumulator; bar_p[2]: tile of P written; bar_pv[2]: its
  // P V done (O_blk ready, that tile of P free); bar_vfree[2]: the same event for the loader of
  // the V^T tiles (every waiter has a barrier of its own, so none can fall two completions
  // behind); bar_ofree[2]: the softmax warps have folded that O_blk into their rows
  __shared__ __align__(8) uint64_t bar_q, bar_k, bar_kfree, bar_v[2], bar_vfree[2], bar_s[2], bar_sfree[2],
      bar_p[2], bar_pv[2], bar_ofree[2];
  constexpr uint32_t TMEM_COLS = WANT_O ? TMEM_COLS_O : TMEM_COLS_A;
  __shared__ uint32_t s_tmem;
  __shared__ int s_fail;
  __shared__ float s_xm[2][2][QT];   // block maxima of the two column halves, double-buffered
  __shared__ float s_xl[2][QT];      // row sums of the two halves

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int bh = b * pa.H + h;
  const int q0 = pa.row0 + qt * QT;                       // position of this tile's first row
  const int q_last = min(pa.row0 + pa.n_rows, q0 + QT) - 1;  // ... and of its last row in use
  const int nkb = q_last / KB + 1;                        // causal: keys up to the last row's position
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sQ = smem_base, sK = smem_base + TILE_B;
  auto sP = [&](int i) { return smem_base + (uint32_t)(2 + (i & 1)) * TILE_B; };
  auto sV = [&](int i) { return smem_base + (uint32_t)(4 + (i & 1)) * TILE_B; };
  const uint32_t id = idesc(pa.bf);

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar_q), 1);
    mbar_init(smem_u32(&bar_k), 1);
    mbar_init(smem_u32(&bar_kfree), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bar_v[i]), 1);
      mbar_init(smem_u32(&bar_vfree[i]), 1);
      mbar_init(smem_u32(&bar_s[i]), 1);
      mbar_init(smem_u32(&bar_sfree[i]), 8);
      mbar_init(smem_u32(&bar_p[i]), 8);
      mbar_init(smem_u32(&bar_pv[i]), 1);
      mbar_init(smem_u32(&bar_ofree[i]), 8);
    }
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&s_tmem)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  auto tmem_s = [&](int i) { return s_tmem + (uint32_t)(i & 1) * 128u; };
  auto tmem_o = [&](int i) { return s_tmem + 256u + (uint32_t)(i & 1) * 128u; };

  // key blocks in the order they are walked: all of them once (WANT_O), or all of them for the
  // row statistics and then those that hold visual columns once more
  const int vb0 = pa.n_sys / KB, vb1 = min(nkb - 1, (pa.n_sys + pa.n_vis - 1) / KB);
  const int n_second = WANT_O ? 0 : max(0, vb1 - vb0 + 1);
  const int n_iter = nkb + n_second;
  auto block_of = [&](int it) { return it < nkb ? it : vb0 + (it - nkb); };

  if (warp == 8) {
    // ---- TMA producer: the key tile of block it + 1 as soon as the scores of block it are
    //      formed, the V^T tile of block it + 1 as soon as P V of block it - 1 is done ----
    if (lane == 0) {
      mbar_expect_tx(smem_u32(&bar_q), TILE_B);
      tma_load_3d(sQ, &mapQ, 0, q0, bh, smem_u32(&bar_q));
      tma_load_3d(sQ + ATOM, &mapQ, 64, q0, bh, smem_u32(&bar_q));
      bool ok = true;
      for (int it = 0; it < n_iter && ok; ++it) {
        const int kb = block_of(it);
        if (it > 0 && !mbar_wait(smem_u32(&bar_kfree), (uint32_t)(it - 1) & 1u)) { ok = false; break; }
        mbar_expect_tx(smem_u32(&bar_k), TILE_B);
        tma_load_3d(sK, &mapK, 0, kb * KB, bh, smem_u32(&bar_k));
        tma_load_3d(sK + ATOM, &mapK, 64, kb * KB, bh, smem_u32(&bar_k));
        if (WANT_O) {
          if (it >= 2 && !mbar_wait(smem_u32(&bar_vfree[it & 1]), ((uint32_t)(it - 2) >> 1) & 1u)) { ok = false; break; }
          mbar_expect_tx(smem_u32(&bar_v[it & 1]), TILE_B);
          tma_load_3d(sV(it), &mapVt, kb * KB, 0, bh, smem_u32(&bar_v[it & 1]));
          tma_load_3d(sV(it) + ATOM, &mapVt, kb * KB + 64, 0, bh, smem_u32(&bar_v[it & 1]));
        }
      }
      if (!ok) s_fail = 1;
    }
  } else if (warp == 9) {
    // ---- MMA issuer: scores one block ahead of the softmax ----
    if (lane == 0) {
      bool ok = mbar_wait(smem_u32(&bar_q), 0);
      auto scores = [&](int it) {   // S[it & 1] = Q K(it)^T
        if (!mbar_wait(smem_u32(&bar_k), (uint32_t)it & 1u)) return false;
        if (it >= 2 && !mbar_wait(smem_u32(&bar_sfree[it & 1]), ((uint32_t)(it - 2) >> 1) & 1u)) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        mma_tile(tmem_s(it), sQ, sK, id);
        umma_commit(smem_u32(&bar_kfree));
        umma_commit(smem_u32(&bar_s[it & 1]));
        return true;
      };
      if (ok) ok = scores(0);
      for (int it = 0; it < n_iter && ok; ++it) {
        if (it + 1 < n_iter) ok = scores(it + 1);
        if (WANT_O && ok) {
          const uint32_t par = ((uint32_t)it >> 1) & 1u;
          if (!mbar_wait(smem_u32(&bar_p[it & 1]), par) || !mbar_wait(smem_u32(&bar_v[it & 1]), par) ||
              (it >= 2 && !mbar_wait(smem_u32(&bar_ofree[it & 1]), ((uint32_t)(it - 2) >> 1) & 1u))) {
            ok = false;
            break;
          }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          mma_tile(tmem_o(it), sP(it), sV(it), id);     // O_blk = P V
          umma_commit(smem_u32(&bar_vfree[it & 1]));
          umma_commit(smem_u32(&bar_pv[it & 1]));
        }
      }
      if (!ok) s_fail = 1;
    }
  } else {
    // ---- warps 0-7: softmax.  Thread = (query row = TMEM lane, column half) ----
    constexpr int HC = KB / 2;                      // columns of a block per thread
    const int row = (warp & 3) * 32 + lane, half = warp >> 2;
    const int qpos = q0 + row;                       // sequence position of this row
    const bool live = qpos <= q_last;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t col0 = (uint32_t)(half * HC);
    float m = -INFINITY, l = 0.f;                    // l: this thread's half of the row sum
    float o[WANT_O ? HC : 1];
    if (WANT_O) {
#pragma unroll
      for (int i = 0; i < HC; ++i) o[i] = 0.f;
    }
    auto pair_sync = [] { asm volatile("bar.sync 1, 256;" ::: "memory"); };
    bool ok = true;
    float inv_l = 0.f;
    float alpha_prev = 1.f;
    // o = o * alpha_j + (P V of block j); alpha_j = 2^(m_{j-1} - m_j) is the factor block j's new
    // maximum put on everything before it
    auto fold = [&](int j, float alpha_j) {
      if (ok && !mbar_wait(smem_u32(&bar_pv[j & 1]), ((uint32_t)j >> 1) & 1u)) ok = false;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
      for (int c = 0; c < HC / 32; ++c) {
        uint32_t r[32];
        tmem_ld32_issue(tmem_o(j) + lane_addr + col0 + (uint32_t)(c * 32), r);
        tmem_wait_ld();
#pragma unroll
        for (int jj = 0; jj < 32; ++jj) o[c * 32 + jj] = fmaf(o[c * 32 + jj], alpha_j, __uint_as_float(r[jj]));
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0)
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar_ofree[j & 1])) : "memory");
    };
    for (int it = 0; it < n_iter; ++it) {
      const int kb = block_of(it);
      const bool second = it >= nkb;
      const uint32_t ts = tmem_s(it) + lane_addr + col0;
      if (!WANT_O && it == nkb) {
        // between the two passes of the probe rows: the whole row sum
        s_xl[half][row] = l;
        pair_sync();
        const float lt = s_xl[0][row] + s_xl[1][row];
        inv_l = (lt > 0.f) ? 1.0f / lt : 0.f;
      }
      // A wait that runs out must not take this thread out of the loop: its partner would wait
      // for it at the pair barrier for ever.  It goes on (on whatever the accumulators hold)
      // without waiting again, and the image is reported at the end.
      if (ok && !mbar_wait(smem_u32(&bar_s[it & 1]), ((uint32_t)it >> 1) & 1u)) ok = false;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int jmax = min(qpos, pa.L - 1) - kb * KB - (int)col0;   // own columns 0 .. jmax are visible
      float alpha = 1.f;
      if (!second) {
        // pass over the block for its maximum: own half, then the partner's through shared memory
        float bm = -INFINITY;
#pragma unroll
        for (int c = 0; c < HC / 32; ++c) {
          uint32_t r[32];
          tmem_ld32_issue(ts + (uint32_t)(c * 32), r);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (c * 32 + j <= jmax) bm = fmaxf(bm, __uint_as_float(r[j]));
        }
        s_xm[it & 1][half][row] = bm;
        pair_sync();
        bm = fmaxf(bm, s_xm[it & 1][half ^ 1][row]);
        const float m_new = fmaxf(m, bm * pa.scale2);
        alpha = (m_new == -INFINITY) ? 1.f : ex2(m - m_new);
        m = m_new;
        l *= alpha;
      }
      if (WANT_O || !second) {
        // probabilities of the own columns (unnormalised), their sum, and, with Z, the tile of P
        float ls = 0.f;
#pragma unroll
        for (int c = 0; c < HC / 32; ++c) {
          uint32_t r[32];
          tmem_ld32_issue(ts + (uint32_t)(c * 32), r);
          tmem_wait_ld();
          float pr[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float e = ex2(fmaf(__uint_as_float(r[j]), pa.scale2, -m));
            pr[j] = (c * 32 + j <= jmax && m != -INFINITY) ? e : 0.f;
            ls += pr[j];
          }
          if (WANT_O) {
            // The half's 64 columns are one swizzle atom of the P tile; chunk ch (8 columns) of
            // the row lies at atom * ATOM + row * 128 + ((ch ^ (row & 7)) * 16).  (P V of the
            // block before, which read this tile, was waited for when its result was folded in.)
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint32_t ch = (uint32_t)(c * 4 + q);
              uint4 v;
              v.x = pack2<T>(pr[q * 8], pr[q * 8 + 1]);
              v.y = pack2<T>(pr[q * 8 + 2], pr[q * 8 + 3]);
              v.z = pack2<T>(pr[q * 8 + 4], pr[q * 8 + 5]);
              v.w = pack2<T>(pr[q * 8 + 6], pr[q * 8 + 7]);
              *reinterpret_cast<uint4*>(smem_gen + (uint32_t)(2 + (it & 1)) * TILE_B + (uint32_t)half * ATOM + (uint32_t)row * 128u +
                                        ((ch ^ ((uint32_t)row & 7u)) << 4)) = v;
            }
          }
        }
        l += ls;
      } else {
        // second pass of the probe rows: normalised probabilities of the block's columns into a
        // staging tile (row-major, 16-bit), from which whole rows leave in runs of 32
        // neighbouring elements per store (a thread owns a row, so storing from the registers
        // would put every lane of a store into a sector of its own)
        uint8_t* stg = smem_gen + 2 * TILE_B;
        if (it > nkb) pair_sync();   // the rows of the block before have left the tile
#pragma unroll
        for (int c = 0; c < HC / 32; ++c) {
          uint32_t r[32];
          tmem_ld32_issue(ts + (uint32_t)(c * 32), r);
          tmem_wait_ld();
          float pr[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float e = ex2(fmaf(__uint_as_float(r[j]), pa.scale2, -m)) * inv_l;
            pr[j] = (c * 32 + j <= jmax) ? e : 0.f;
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint4 v;
            v.x = pack2<T>(pr[q * 8], pr[q * 8 + 1]);
            v.y = pack2<T>(pr[q * 8 + 2], pr[q * 8 + 3]);
            v.z = pack2<T>(pr[q * 8 + 4], pr[q * 8 + 5]);
            v.w = pack2<T>(pr[q * 8 + 6], pr[q * 8 + 7]);
            *reinterpret_cast<uint4*>(stg + (uint32_t)row * STG_ROW + (col0 + (uint32_t)(c * 32 + q * 8)) * 2u) = v;
          }
        }
        pair_sync();
        {
          const int x0 = kb * KB - pa.n_sys;   // visual index of the block's first column
          for (int rr = warp; rr < QT; rr += 8) {
            const int qp = q0 + rr;
            if (qp > q_last) break;
            T* drow = out + (((size_t)bh * pa.n_rows + (qp - pa.row0)) * pa.n_vis);
            const T* srow = reinterpret_cast<const T*>(stg + (uint32_t)rr * STG_ROW);
#pragma unroll
            for (int j = 0; j < KB / 32; ++j) {
              const int col = lane + 32 * j, x = x0 + col;
              if (x >= 0 && x < pa.n_vis) drow[x] = srow[col];
            }
          }
        }
      }
      // this score accumulator may be overwritten
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0)
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar_sfree[it & 1])) : "memory");
      if (WANT_O) {
        // hand this block's P to the tensor core, then fold the P V of the block BEFORE into the
        // own half of the row of Z: that product ran while this block's probabilities were
        // formed (two tiles of P, two accumulators for P V), so the wait below is short
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0)
          asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar_p[it & 1])) : "memory");
        if (it > 0) fold(it - 1, alpha_prev);
        alpha_prev = alpha;
      }
    }
    if (WANT_O && n_iter > 0) fold(n_iter - 1, alpha_prev);
    if (WANT_O) {
      // the whole row sum (every thread of the team comes here, whatever happened above)
      s_xl[half][row] = l;
      pair_sync();
      const float lt = s_xl[0][row] + s_xl[1][row];
      inv_l = (lt > 0.f) ? 1.0f / lt : 0.f;
    }
    if (!ok) s_fail = 1;
    if (WANT_O) {
      // The rows of Z leave through a row-major staging tile in the first tile of P (every P V
      // has completed): a thread owns half a row, so stores from its registers would put each
      // lane of a store into a sector of its own; from the tile a warp writes a row per store.
      uint8_t* stg = smem_gen + 2 * TILE_B;
#pragma unroll
      for (int q = 0; q < HC / 8; ++q) {
        uint4 v;
        v.x = pack2<T>(o[q * 8] * inv_l, o[q * 8 + 1] * inv_l);
        v.y = pack2<T>(o[q * 8 + 2] * inv_l, o[q * 8 + 3] * inv_l);
        v.z = pack2<T>(o[q * 8 + 4] * inv_l, o[q * 8 + 5] * inv_l);
        v.w = pack2<T>(o[q * 8 + 6] * inv_l, o[q * 8 + 7] * inv_l);
        *reinterpret_cast<uint4*>(stg + (uint32_t)row * STG_ROW + (uint32_t)(half * HC + q * 8) * 2u) = v;
      }
    }
    pair_sync();
    if (s_fail == 0) {
      if (WANT_O) {
        uint8_t* stg = smem_gen + 2 * TILE_B;
        for (int rr = warp; rr < QT; rr += 8) {
          const int qp = q0 + rr;
          if (qp > q_last) break;
          // row qp - n_sys of O, columns h * dh ..: 256 bytes, 8 per lane
          uint2* dst = reinterpret_cast<uint2*>(out + (((size_t)b * pa.n_vis + (qp - pa.n_sys)) * pa.H + h) * DH);
          dst[lane] = *reinterpret_cast<const uint2*>(stg + (uint32_t)rr * STG_ROW + (uint32_t)lane * 8u);
        }
      }
    } else if (status != nullptr && threadIdx.x == 0) {
      atomicMax(&status[b], (int)TC_ERR_CUDA);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 9) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(s_tmem),
                 "r"(TMEM_COLS)
                 : "memory");
  }
}

// Vt [BH][dh][Lp] = V [BH][L][dh]^T, columns L .. Lp - 1 zero (Lp and dh even).  64 x 64 tiles,
// two elements per access: a warp reads and writes 128 contiguous bytes.  grid (Lp / 64 rounded
// up, dh / 64 rounded up, BH), block (32, 8).
template <typename T>
__global__ void __launch_bounds__(256) transpose_v_kernel(const T* __restrict__ V, T* __restrict__ Vt,
                                                         int L, int Lp, int dh) {
  __shared__ T t[64][66];
  const size_t bh = blockIdx.z;
  const int l0 = blockIdx.x * 64, d0 = blockIdx.y * 64;
  const int tx = threadIdx.x, ty = threadIdx.y;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int l = l0 + ty + 8 * i, d = d0 + 2 * tx;
    uint32_t v = 0u;
    if (l < L && d < dh) v = *reinterpret_cast<const uint32_t*>(V + (bh * L + l) * dh + d);
    *reinterpret_cast<uint32_t*>(&t[ty + 8 * i][2 * tx]) = v;
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int dd = ty + 8 * i, d = d0 + dd, l = l0 + 2 * tx;
    if (d < dh && l < Lp) {
      T pair[2] = {t[2 * tx][dd], t[2 * tx + 1][dd]};
      *reinterpret_cast<uint32_t*>(Vt + (bh * dh + d) * Lp + l) = *reinterpret_cast<uint32_t*>(pair);
    }
  }
}

// [inner, rows, BH] 16-bit tensor, box 64 x 128 x 1, 128-byte swizzle, zero fill
bool encode16(CUtensorMap* map, const void* base, int inner, int rows, int bh, int bf) {
  encode_fn enc = get_encode();
  if (enc == nullptr) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)rows, (cuuint64_t)bh};
  const cuuint64_t strides[2] = {(cuuint64_t)inner * 2, (cuuint64_t)rows * inner * 2};
  const cuuint32_t box[3] = {64, 128, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return enc(map, bf ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3,
             const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename T>
tc_status run_probe(int B, int H, int L, int n_sys, int n_vis, int probe_start, int n_probe,
                    const void* Q, const void* K, const void* V, void* O, void* A, void* Vt, int Lp,
                    int32_t* status, cudaStream_t st, int bf) {
  CUtensorMap mq, mk, mv;
  if (!encode16(&mq, Q, DH, L, B * H, bf) || !encode16(&mk, K, DH, L, B * H, bf)) return TC_ERR_CUDA;
  if (O != nullptr && !encode16(&mv, Vt, Lp, DH, B * H, bf)) return TC_ERR_CUDA;
  if (O == nullptr) mv = mk;
  if (cudaFuncSetAttribute((const void*)probe_kernel<T, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)SMEM_O) != cudaSuccess ||
      cudaFuncSetAttribute((const void*)probe_kernel<T, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)SMEM_A) != cudaSuccess)
    return TC_ERR_CUDA;
  ProbeArgs pa;
  pa.L = L; pa.n_sys = n_sys; pa.n_vis = n_vis; pa.H = H;
  pa.scale2 = 1.4426950408889634f / sqrtf((float)DH);
  pa.bf = bf;
  if (O != nullptr) {
    Scope scope_(KC_GRAM, st);
    dim3 tg((Lp + 63) / 64, (DH + 63) / 64, B * H), tb(32, 8);
    transpose_v_kernel<T><<<tg, tb, 0, st>>>((const T*)V, (T*)Vt, L, Lp, DH);
    note_launch();
    pa.row0 = n_sys; pa.n_rows = n_vis;
    dim3 grid((n_vis + QT - 1) / QT, H, B);
    probe_kernel<T, true><<<grid, 320, SMEM_O, st>>>(mq, mk, mv, pa, (T*)O, status);
    note_launch();
  }
  if (A != nullptr && n_probe > 0) {
    Scope scope_(KC_ATTN, st);
    // columns a probe row may not see (keys after it) are never visited: they read as zero
    if (cudaMemsetAsync(A, 0, (size_t)B * H * n_probe * n_vis * sizeof(T), st) != cudaSuccess) return TC_ERR_CUDA;
    pa.row0 = probe_start; pa.n_rows = n_probe;
    dim3 grid((n_probe + QT - 1) / QT, H, B);
    probe_kernel<T, false><<<grid, 320, SMEM_A, st>>>(mq, mk, mv, pa, (T*)A, status);
    note_launch();
  }
  return TC_OK;
}

}  // namespace

size_t probe_workspace_bytes(int B, int H, int L, int dh) {
  const size_t Lp = (size_t)(L + 7) / 8 * 8;
  return align_up((size_t)B * H * dh * Lp * 2, 256);
}

tc_status launch_probe(int B, int H, int dh, int L, int n_sys, int n_vis, int probe_start, int n_probe,
                       const void* Q, const void* K, const void* V, void* O, void* A, void* ws,
                       int32_t* status, cudaStream_t st, int bf) {
  if (dh != DH) return TC_ERR_UNSUPPORTED;
  const int Lp = (L + 7) / 8 * 8;
  if (bf)
    return run_probe<__nv_bfloat16>(B, H, L, n_sys, n_vis, probe_start, n_probe, Q, K, V, O, A, ws, Lp,
                                    status, st, 1);
  return run_probe<__half>(B, H, L, n_sys, n_vis, probe_start, n_probe, Q, K, V, O, A, ws, Lp, status, st, 0);
}

}  // namespace tc
