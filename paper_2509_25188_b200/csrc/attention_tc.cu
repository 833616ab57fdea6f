// Bidirectional (non-causal) multi-head attention on the 5th-generation tensor cores, head size 128.
// Flash style: one pass over the keys in tiles of 128 with a running row max and row sum, so the
// [queries x keys] scores never leave the SM.  Every query of a sequence sees keys [0, kv_len) of
// that sequence: there is no mask, only the ragged tail of the last key tile.
//
// One CTA = 128 query rows of one head.  Per key tile j
//     S_j  = Q K_j^T            tcgen05.mma, Q and K_j K-major in shared memory (TMA, 128-byte swizzle),
//                               fp32 scores in tensor memory (two buffers)
//     P_j  = exp2(S_j c - m)    by the softmax warps, written as packed bf16 pairs to tensor memory
//                               (two buffers), where the second product reads it as its A operand
//     O   += P_j V_j            tcgen05.mma, A from tensor memory, V_j read MN-major from shared memory
//                               (rows of V are keys = the K dimension); O stays in tensor memory for
//                               the whole pass.
// m is the reference maximum the probabilities are taken against.  It follows the running row
// maximum lazily: only when the maximum has grown by more than 8 (a factor 256) do the softmax
// threads rescale O and the row sum; the quotient O / l at the end does not depend on m.
//
// Warp roles (352 threads): 0 = TMA producer, 1 = issues the S products (owns tensor memory),
// 2 = issues the P V products, 3-10 = softmax and output: thread (row, half) handles 64 of the 128
// columns of its row (keys of S, head dimensions of O), the two halves exchanging their row maxima
// through shared memory.  The two products have separate issuing threads because one thread issues
// at most one tcgen05.mma per ~132 cycles while an N = 128 instruction occupies the pipe for 64.
// Tensor memory (512 columns): S buffers at 0 and 128, O at 256, P buffers at 384 and 448.
// Every wait is bounded; a wait that runs out sets the status word and the CTA leaves normally.
#include <math.h>

#include "common.cuh"
#include "ptx.cuh"

namespace l2pd {

namespace {

constexpr int BQ = 128, BKV = 128, DH = 128;
constexpr uint32_t HALF_BYTES = 128 * 128;        // 128 rows x 64 bf16: one swizzled half tile
constexpr uint32_t TILE_BYTES = 2 * HALF_BYTES;   // 128 x 128 bf16
constexpr int SMEM_BYTES = 5 * TILE_BYTES + 1024; // Q, 2 x K, 2 x V (+ alignment slack)

struct AttnTcParams {
  bf16 *out;
  const SeqMeta *meta;
  SeqMeta single;
  int use_single;
  int64_t out_stride;
  float scale_log2;
  int kv_rows_per_seq;   // rows between two sequences in the key/value tensor maps
  int kv_row_base;       // first row of this layer's store in the key/value tensor maps
  int kv_packed;         // keys / values are the packed activation rows: row = row0 of the sequence + key
  int32_t *status;
};

enum { B_QFULL = 0, B_KFULL = 1, B_VFULL = 3, B_KEMPTY = 5, B_VEMPTY = 7, B_SFULL = 9, B_SEMPTY = 11,
       B_PFULL = 13, B_PVDONE = 15, B_XCHG = 17, B_COUNT = 18 };
constexpr int N_SOFTMAX_WARPS = 8;
constexpr float RESCALE_STEP = 8.0f;   // log2 units the row maximum may run ahead of the reference maximum

__device__ __forceinline__ void fail(int32_t *status, int code) {
  if (status) atomicCAS(status, 0, code);
}

__global__ void __launch_bounds__(352, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const AttnTcParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[B_COUNT];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ float xchg[2][2][BQ];   // [parity of the tile][column half][row]: row maxima, then row sums

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = base, sK = base + TILE_BYTES, sV = base + 3 * TILE_BYTES;
  const uint32_t bar0 = ptx::smem_u32(bars);
  auto bar = [&](int i) { return bar0 + 8u * i; };

  if (threadIdx.x == 0) {
    ptx::mbar_init(bar(B_QFULL), 1);
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(bar(B_KFULL + b), 1); ptx::mbar_init(bar(B_VFULL + b), 1);
      ptx::mbar_init(bar(B_KEMPTY + b), 1); ptx::mbar_init(bar(B_VEMPTY + b), 1);
      ptx::mbar_init(bar(B_SFULL + b), 1); ptx::mbar_init(bar(B_SEMPTY + b), N_SOFTMAX_WARPS);
      ptx::mbar_init(bar(B_PFULL + b), N_SOFTMAX_WARPS); ptx::mbar_init(bar(B_PVDONE + b), 1);
    }
    ptx::mbar_init(bar(B_XCHG), N_SOFTMAX_WARPS);
    abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&tmQ); ptx::prefetch_tensormap(&tmK); ptx::prefetch_tensormap(&tmV);
  }
  if (warp == 1) { ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), 512); ptx::tmem_relinquish(); }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = tmem_slot;
  const uint32_t tS = tmem_base, tO = tmem_base + 256, tP = tmem_base + 384;
  grid_dep_launch();
  grid_dep_wait();

  const SeqMeta m = p.use_single ? p.single : p.meta[blockIdx.z];
  const int q0 = blockIdx.x * BQ;
  const int h = blockIdx.y;
  const int kv_len = m.kv_len;
  const bool live = q0 < m.n_rows;                 // uniform over the CTA
  const int n_tiles = live ? (kv_len + BKV - 1) / BKV : 0;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && live) {
      const uint64_t pol = ptx::policy_evict_last();   // K and V of a head are re-read by every query tile
      bool ok = true;
      ptx::mbar_arrive_expect_tx(bar(B_QFULL), TILE_BYTES);
      ptx::tma_load_2d_hint(sQ, &tmQ, bar(B_QFULL), h * DH, m.row0 + q0, pol);
      ptx::tma_load_2d_hint(sQ + HALF_BYTES, &tmQ, bar(B_QFULL), h * DH + 64, m.row0 + q0, pol);
      const int krow = p.kv_row_base + (p.kv_packed ? m.row0 : m.seq * p.kv_rows_per_seq);
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int st = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        if (!ptx::mbar_wait(bar(B_KEMPTY + st), ph ^ 1u)) { fail(p.status, DEV_TIMEOUT_PRODUCER); ok = false; break; }
        ptx::mbar_arrive_expect_tx(bar(B_KFULL + st), TILE_BYTES);
        ptx::tma_load_2d_hint(sK + st * TILE_BYTES, &tmK, bar(B_KFULL + st), h * DH, krow + j * BKV, pol);
        ptx::tma_load_2d_hint(sK + st * TILE_BYTES + HALF_BYTES, &tmK, bar(B_KFULL + st), h * DH + 64, krow + j * BKV, pol);
        if (!ptx::mbar_wait(bar(B_VEMPTY + st), ph ^ 1u)) { fail(p.status, DEV_TIMEOUT_PRODUCER); ok = false; break; }
        ptx::mbar_arrive_expect_tx(bar(B_VFULL + st), TILE_BYTES);
        ptx::tma_load_2d_hint(sV + st * TILE_BYTES, &tmV, bar(B_VFULL + st), h * DH, krow + j * BKV, pol);
        ptx::tma_load_2d_hint(sV + st * TILE_BYTES + HALF_BYTES, &tmV, bar(B_VFULL + st), h * DH + 64, krow + j * BKV, pol);
      }
      if (!ok) abort_flag = 1;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ S_j = Q K_j^T
    if (lane == 0 && live) {
      const uint32_t idesc = ptx::idesc_bf16(BQ, BKV);
      bool ok = ptx::mbar_wait(bar(B_QFULL), 0);
      if (!ok) fail(p.status, DEV_TIMEOUT_MMA);
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int st = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        if (!ptx::mbar_wait(bar(B_KFULL + st), ph) || !ptx::mbar_wait(bar(B_SEMPTY + st), ph ^ 1u)) {
          fail(p.status, DEV_TIMEOUT_MMA); ok = false; break;
        }
        ptx::tc_fence_after_sync();
#pragma unroll
        for (int k = 0; k < DH / 16; ++k) {
          const uint64_t a = ptx::smem_desc_sw128(sQ + (k >> 2) * HALF_BYTES) + 2u * (k & 3);
          const uint64_t b = ptx::smem_desc_sw128(sK + st * TILE_BYTES + (k >> 2) * HALF_BYTES) + 2u * (k & 3);
          ptx::mma_bf16_ss(tS + st * BKV, a, b, idesc, k ? 1u : 0u);
        }
        ptx::mma_commit(bar(B_KEMPTY + st));
        ptx::mma_commit(bar(B_SFULL + st));
      }
      if (!ok) abort_flag = 1;
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ O += P_j V_j
    if (lane == 0 && live) {
      const uint32_t idesc = ptx::idesc_bf16_b_mn(BQ, DH);
      bool ok = true;
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int st = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        if (!ptx::mbar_wait(bar(B_VFULL + st), ph) || !ptx::mbar_wait(bar(B_PFULL + st), ph)) {
          fail(p.status, DEV_TIMEOUT_MMA); ok = false; break;
        }
        ptx::tc_fence_after_sync();
#pragma unroll
        for (int k = 0; k < BKV / 16; ++k) {   // 16 keys per instruction: 8 columns of P, two 8-row groups of the V tile
          const uint64_t b = ptx::smem_desc_sw128_mn(sV + st * TILE_BYTES + k * 2048, HALF_BYTES);
          ptx::mma_bf16_ts(tO, tP + st * 64 + k * 8, b, idesc, (j > 0 || k > 0) ? 1u : 0u);
        }
        ptx::mma_commit(bar(B_VEMPTY + st));
        ptx::mma_commit(bar(B_PVDONE + st));
      }
      if (!ok) abort_flag = 1;
    }
  } else if (live) {
    // ------------------------------------------------------------------ softmax and output
    const int q = warp & 3, hf = (warp - 3) >> 2;
    const int row = q * 32 + lane;
    const uint32_t lane_base = (uint32_t)(q * 32) << 16;
    const float c = p.scale_log2;
    float m_ref = -INFINITY, l_run = 0.f;
    bool ok = true;
    uint32_t r[64];

    // meeting point of the eight softmax warps (bounded, unlike bar.sync): use number u completes phase u
    auto meet = [&](int u) -> bool {
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar(B_XCHG));
      return ptx::mbar_wait(bar(B_XCHG), u & 1);
    };

    for (int j = 0; j < n_tiles && ok; ++j) {
      const int st = j & 1;
      const uint32_t ph = (j >> 1) & 1;
      if (!ptx::mbar_wait(bar(B_SFULL + st), ph)) { ok = false; break; }
      ptx::tc_fence_after_sync();
      ptx::tmem_ld_x32(tS + lane_base + st * BKV + hf * 64, r);
      ptx::tmem_ld_x32(tS + lane_base + st * BKV + hf * 64 + 32, r + 32);
      ptx::tmem_ld_wait();
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar(B_SEMPTY + st));       // the scores are in registers: S buffer free
      const int n_valid = kv_len - j * BKV - hf * 64;            // this thread's columns that are keys
      if (n_valid < 64) {                                        // ragged last tile only
#pragma unroll
        for (int i = 0; i < 64; ++i) if (i >= n_valid) r[i] = 0xff800000u;   // -inf
      }
      float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int i = 0; i < 64; i += 4) {
#pragma unroll
        for (int e = 0; e < 4; ++e) mx[e] = fmaxf(mx[e], __uint_as_float(r[i + e]));
      }
      float mxx = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
      xchg[st][hf][row] = mxx;
      if (!meet(j)) { ok = false; break; }
      mxx = fmaxf(mxx, xchg[st][hf ^ 1][row]);
      const float m_new = fmaxf(m_ref, mxx * c);
      const bool rescale = m_new > m_ref + RESCALE_STEP;             // first tile: m_ref = -inf
      const float factor = rescale ? ptx::ex2(m_ref - m_new) : 1.0f; // first tile: 0
      if (rescale) m_ref = m_new;
      // probabilities, packed two to a column
      float rs[4] = {0.f, 0.f, 0.f, 0.f};
      const float neg_m = -m_ref;
#pragma unroll
      for (int i = 0; i < 64; i += 2) {
        const float p0 = ptx::ex2(fmaf(__uint_as_float(r[i]), c, neg_m));
        const float p1 = ptx::ex2(fmaf(__uint_as_float(r[i + 1]), c, neg_m));
        rs[(i >> 1) & 3] += p0 + p1;
        __nv_bfloat162 t = __floats2bfloat162_rn(p0, p1);
        r[i >> 1] = *reinterpret_cast<uint32_t *>(&t);
      }
      l_run = fmaf(l_run, factor, (rs[0] + rs[1]) + (rs[2] + rs[3]));
      // P buffer st was last read by the product of tile j - 2; O is at rest once that of tile j - 1 is done
      if (j >= 2 && !ptx::mbar_wait(bar(B_PVDONE + st), ph ^ 1u)) { ok = false; break; }
      ptx::tc_fence_after_sync();
      ptx::tmem_st_x32(tP + lane_base + st * 64 + hf * 32, r);
      // tensor-memory loads and stores are warp-wide instructions: if any row of the warp moves its
      // reference maximum, the whole warp rewrites its rows of O (rows that keep theirs scale by 1)
      if (__any_sync(0xffffffffu, rescale && j > 0)) {
        // bring this thread's 64 columns of O to the new reference maximum
        if (!ptx::mbar_wait(bar(B_PVDONE + (st ^ 1)), ((j - 1) >> 1) & 1)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        ptx::tmem_ld_x32(tO + lane_base + hf * 64, r + 32);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 32; i < 64; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * factor);
        ptx::tmem_st_x32(tO + lane_base + hf * 64, r + 32);
        ptx::tmem_st_wait();
        ptx::tmem_ld_x32(tO + lane_base + hf * 64 + 32, r + 32);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 32; i < 64; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * factor);
        ptx::tmem_st_x32(tO + lane_base + hf * 64 + 32, r + 32);
      }
      ptx::tmem_st_wait();
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar(B_PFULL + st));
    }
    if (ok) ok = ptx::mbar_wait(bar(B_PVDONE + ((n_tiles - 1) & 1)), ((n_tiles - 1) >> 1) & 1);
    if (ok) {
      ptx::tc_fence_after_sync();
      ptx::tmem_ld_x32(tO + lane_base + hf * 64, r);
      ptx::tmem_ld_x32(tO + lane_base + hf * 64 + 32, r + 32);
      const int xs = n_tiles & 1;                        // a slot the last tile's maxima did not use
      xchg[xs][hf][row] = l_run;
      ok = meet(n_tiles);
      const float inv = 1.0f / (l_run + xchg[xs][hf ^ 1][row]);
      ptx::tmem_ld_wait();
      if (ok && q0 + row < m.n_rows) {
        bf16 *og = p.out + (int64_t)(m.row0 + q0 + row) * p.out_stride + h * DH + hf * 64;
#pragma unroll
        for (int i = 0; i < 64; i += 8) {
          uint4 pk;
          uint32_t *pw = reinterpret_cast<uint32_t *>(&pk);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 t = __floats2bfloat162_rn(__uint_as_float(r[i + 2 * e]) * inv, __uint_as_float(r[i + 2 * e + 1]) * inv);
            pw[e] = *reinterpret_cast<uint32_t *>(&t);
          }
          *reinterpret_cast<uint4 *>(og + i) = pk;
        }
      }
    }
    if (!ok) { fail(p.status, DEV_TIMEOUT_EPILOGUE); abort_flag = 1; }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (abort_flag) {
    // A wait ran out: give copies still in flight time to land before the CTA's shared memory goes away.
    const uint64_t t0 = ptx::globaltimer();
    while (ptx::globaltimer() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

bool attention_tc_supported(int dh, int64_t q_stride, int64_t kv_row_stride, int64_t out_stride) {
  return dh == DH && (q_stride % 8) == 0 && (kv_row_stride % 8) == 0 && (out_stride % 8) == 0;
}

cudaError_t launch_attention_tc(cudaStream_t st, const TmaDesc &tq, const TmaDesc &tk, const TmaDesc &tv,
                                const SeqMeta *meta, bf16 *out, int64_t out_stride, int kv_rows_per_seq,
                                int kv_row_base, int kv_packed, int n_slots, int max_q_rows, int H, int32_t *status) {
  AttnTcParams p;
  p.out = out; p.meta = meta; p.use_single = 0; p.out_stride = out_stride;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
  p.kv_rows_per_seq = kv_rows_per_seq; p.kv_row_base = kv_row_base; p.kv_packed = kv_packed; p.status = status;
  if (meta == nullptr) {
    // stand-alone call: one sequence, max_q_rows queries, n_slots carries the key count
    p.use_single = 1;
    p.single.seq = 0; p.single.row0 = 0; p.single.n_rows = max_q_rows; p.single.pos0 = 0;
    p.single.kv_len = n_slots; p.single.blk_start = 0; p.single.n_blk_rows = 0; p.single.block = 0;
    n_slots = 1;
  }
  if (max_q_rows <= 0 || n_slots <= 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (e != cudaSuccess) return e;
  dim3 grid(ceil_div(max_q_rows, BQ), H, n_slots);
  return launch_kernel(attention_tc_kernel, grid, dim3(352), (size_t)SMEM_BYTES, st, tq.map, tk.map, tv.map, p);
}

}  // namespace l2pd
