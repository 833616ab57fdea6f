// bf16 GEMM on the 5th-generation tensor cores:  acc[M,N] = A[M,K] * W[N,K]^T, fp32 accumulation
// in tensor memory, operands brought to shared memory by TMA (128-byte swizzle), one thread
// issuing tcgen05.mma, four warps draining the accumulator.  Persistent CTAs (one per SM) walk
// the output tiles; the accumulator is double-buffered in TMEM so a tile's epilogue overlaps the
// next tile's main loop.
//
// Epilogues
//   EPI_STORE     C (bf16)  = acc                                   plain projection
//   EPI_QKV_ROPE  C (bf16)  = acc, the q and k columns rotated by the row's position (RoPE): QKV
//                 projection whose weight rows were reordered so that a rotary pair is two adjacent columns
//   EPI_RESIDUAL  X (fp32) += acc                                   output / down projection
//   EPI_SWIGLU    H (bf16)  = silu(acc_gate) * acc_up               gate/up projection; the B tile
//                 holds tile_n/2 rows of W_gate followed by tile_n/2 rows of W_up
//   EPI_LMHEAD    per-row running (max, sum exp, argmax) over the vocabulary tile, written as one
//                 record per (tile, row): the logits are never stored (Eq. 3-4 need only these).
//
// Warp roles: warp 0 = TMA producer of the weight tiles, warp 1 = TMEM owner and MMA issuer,
// warp 2 = second MMA issuer (two-slab units only), warps 3-6 (and 7-10 for the second slab) =
// epilogue (warp w reads TMEM lanes 32*(w%4) .. +31), last warp = TMA producer of the activation
// tiles.  The loads have two issuing threads because one thread needs ~170 cycles per TMA
// instruction, and a k-block of a two-slab unit takes three of them plus an L2 prefetch; the weight
// producer depends on no earlier kernel and starts while the previous kernel is still running.
//
// One thread can issue a tcgen05.mma (K = 16) only every ~132 cycles, whatever its N, while the
// tensor pipe needs N/2 cycles for it: a single issuer keeps the pipe busy only for N = 256.
// A unit of two row slabs has two independent accumulators, each fed by its own issuing thread,
// so the pipe sees two instructions per 132 cycles and stays busy for any N >= 132.
#include <math.h>
#include <stdio.h>

#include "common.cuh"
#include "gemm_device.cuh"
#include "ptx.cuh"

namespace l2pd {

using namespace gemm_dev;

namespace {

// CG = 1: one CTA per 128 x tile_n output tile.
// CG = 2: a cluster of two CTAs per 256 x tile_n tile (cta_group::2).  CTA r loads A rows
//         [128 r, 128 r + 128) and the r-th half of the B tile (for SwiGLU: CTA 0 the gate rows,
//         CTA 1 the up rows), so each SM takes in half of the weight tile; the leader CTA (rank 0)
//         issues the MMAs, which read both CTAs' shared memory and write both CTAs' tensor memory.
//         All load-completion bytes are counted on the leader's `full` barriers; `empty` and
//         `tmem full` are signalled in both CTAs by a multicast commit; the peer's epilogue warps
//         release the accumulator on the leader's `tmem empty` barrier.
template <int EPI, int CG>
__device__ __forceinline__ void gemm_body(const CUtensorMap *tmA, const CUtensorMap *tmB, const CUtensorMap *tmB2,
                                          const CUtensorMap *tmC, const KParams &p, uint8_t *smem_raw, uint64_t *bars, uint32_t *tmem_slot,
                                          int *abort_flag) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = (CG == 2) ? ptx::cluster_ctarank() : 0u;
  const bool leader = rank == 0;
  const int group = (CG == 2) ? (blockIdx.x >> 1) : blockIdx.x;
  const int n_groups = (CG == 2) ? (gridDim.x >> 1) : gridDim.x;

  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = base;
  const uint32_t sB = base + p.n_stages * p.a_stage_bytes;
  const uint32_t sOut = sA + (uint32_t)(p.n_stages - 2) * p.a_stage_bytes;   // output staging: see drain_tile_staged
  const int slabs = p.slabs;
  const int nbuf = (slabs == 1 && !p.kil) ? 2 : 1;   // accumulator buffers a unit can alternate between
  const int unit_rows = TILE_M * CG * slabs;
  const uint32_t bar0 = ptx::smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (MAX_STAGES + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * MAX_STAGES + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * MAX_STAGES + 2 + b); };
  const uint32_t sfree_bar = bar0 + 8u * (2 * MAX_STAGES + 4);

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.n_stages; ++s) { ptx::mbar_init(full_bar(s), 1); ptx::mbar_init(empty_bar(s), slabs); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(tfull_bar(b), p.kil ? 2 : slabs); ptx::mbar_init(tempty_bar(b), 4 * CG * slabs); }
    ptx::mbar_init(sfree_bar, 4 * slabs);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(tmA);
    ptx::prefetch_tensormap(tmB);
    if (EPI == EPI_SWIGLU) ptx::prefetch_tensormap(tmB2);
    if (EPI != EPI_LMHEAD && p.out_tma) ptx::prefetch_tensormap(tmC);
  }
  if (warp == 1) {
    if (CG == 2) { ptx::tmem_alloc_pair(ptx::smem_u32(tmem_slot), TMEM_COLS); ptx::tmem_relinquish_pair(); }
    else { ptx::tmem_alloc(ptx::smem_u32(tmem_slot), TMEM_COLS); ptx::tmem_relinquish(); }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (CG == 2) ptx::cluster_sync();     // the peer's barriers exist before anything arrives on them
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // The set-up above overlaps the previous kernel's tail.  Of what follows, only the activation loads
  // (producer) and the output stores (epilogue warps) touch memory that other kernels of the stream
  // write or read: those threads call grid_dep_wait() themselves, after the producer has already
  // requested the first weight tiles, which no kernel writes.
  grid_dep_launch();

  const int num_units = p.m_tiles * p.n_tiles * p.k_splits;
  const int num_kb = (p.K + TILE_K - 1) / TILE_K;
  const int kb_per = (num_kb + p.k_splits - 1) / p.k_splits;
  const int half_n = p.tile_n >> 1;
  // unit -> (row tile, column tile, K slice).  Within a K slice the units run group by group of
  // group_m row tiles; inside a group the row tiles of one column tile are adjacent, then the next
  // column tile follows.  The CTAs running at the same time thus share a few weight tiles, and a
  // group's activation rows (sized to a fraction of L2) stay resident while its column tiles stream by.
  int unit_ks = 0;   // K slice of the unit decoded last
  auto decode = [&](int u, int &mt, int &nt, int &kb0, int &kb1) {
    const int per_slice = p.m_tiles * p.n_tiles;
    const int ks = u / per_slice;
    unit_ks = ks;
    const int r = u - ks * per_slice;
    const int per_group = p.group_m * p.n_tiles;
    const int g = r / per_group;
    const int w = r - g * per_group;
    const int gm = min(p.group_m, p.m_tiles - g * p.group_m);   // the last group may be smaller
    nt = w / gm;
    mt = g * p.group_m + (w - nt * gm);
    kb0 = ks * kb_per;
    kb1 = min(num_kb, kb0 + kb_per);
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const uint64_t pol_w = ptx::policy_evict_first();   // weights are read once per step
      const uint32_t b_bytes = (CG == 2) ? (uint32_t)half_n * 128u : (uint32_t)p.tile_n * 128u;
      const uint32_t tx = (CG == 2 ? (1 + p.a_peer_loads) : 1) * (uint32_t)slabs * p.a_box_bytes + CG * b_bytes;
      auto issue_b = [&](int stage, int kb, int nt) {   // weight tile of k-block kb (and the stage's byte count)
        const uint32_t dstB = sB + stage * p.b_stage_bytes;
        if (CG == 1) {
          ptx::mbar_arrive_expect_tx(full_bar(stage), tx);
          if (EPI == EPI_SWIGLU) {
            ptx::tma_load_2d_hint(dstB, tmB, full_bar(stage), kb * TILE_K, nt * half_n, pol_w);
            ptx::tma_load_2d_hint(dstB + half_n * 128, tmB2, full_bar(stage), kb * TILE_K, nt * half_n, pol_w);
          } else {
            ptx::tma_load_2d_hint(dstB, tmB, full_bar(stage), kb * TILE_K, nt * p.tile_n, pol_w);
          }
        } else {
          if (leader) ptx::mbar_arrive_expect_tx(full_bar(stage), tx);
          const uint32_t lead_full = ptx::mapa(full_bar(stage), 0);
          if (EPI == EPI_SWIGLU)
            ptx::tma_load_2d_pair_hint(dstB, leader ? tmB : tmB2, lead_full, kb * TILE_K, nt * half_n, pol_w);
          else
            ptx::tma_load_2d_pair_hint(dstB, tmB, lead_full, kb * TILE_K, nt * p.tile_n + (int)rank * half_n, pol_w);
        }
      };
      // Weights come from HBM exactly once and the ring holds only a few k-blocks, fewer than HBM's latency
      // under load is worth: the tile PF_AHEAD k-blocks further on is asked into L2 with every load.
      constexpr int PF_AHEAD = 8;
      auto prefetch_b = [&](int kb, int nt) {
        if (EPI == EPI_LMHEAD) return;   // HBM-bound already: asking tiles into L2 early only adds re-reads (measured +15 % traffic)
        if (CG == 1) {
          if (EPI == EPI_SWIGLU) {
            ptx::tma_prefetch_l2_2d(tmB, kb * TILE_K, nt * half_n);
            ptx::tma_prefetch_l2_2d(tmB2, kb * TILE_K, nt * half_n);
          } else {
            ptx::tma_prefetch_l2_2d(tmB, kb * TILE_K, nt * p.tile_n);
          }
        } else if (EPI == EPI_SWIGLU) {
          ptx::tma_prefetch_l2_2d(leader ? tmB : tmB2, kb * TILE_K, nt * half_n);
        } else {
          ptx::tma_prefetch_l2_2d(tmB, kb * TILE_K, nt * p.tile_n + (int)rank * half_n);
        }
      };
      // one producer thread for the weights (this warp), one for the activations (last warp): both walk the
      // same units, k-blocks and stages; every unit starts at stage 0 (so the staging area is what a unit
      // fills last), with one phase bit per stage.  No kernel writes weights, so this thread does not wait
      // for the previous kernel of the stream.
      uint32_t phases = 0;
      int lt = 0;
      bool ok = true;
      for (int u = group; u < num_units && ok; u += n_groups, ++lt) {
        int mt, nt, kb0, kb1;
        decode(u, mt, nt, kb0, kb1);
        int stage = 0;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (kb + p.n_stages + PF_AHEAD < kb1) prefetch_b(kb + p.n_stages + PF_AHEAD, nt);
          if (p.gate && lt > 0 && kb - kb0 == p.n_stages - 2 &&
              !ptx::mbar_wait(sfree_bar, (uint32_t)(lt - 1) & 1u)) { fail(p.status, DEV_TIMEOUT_PRODUCER); ok = false; break; }
          if (!ptx::mbar_wait(empty_bar(stage), ((phases >> stage) & 1u) ^ 1u)) { fail(p.status, DEV_TIMEOUT_PRODUCER); ok = false; break; }
          issue_b(stage, kb, nt);
          if (kb - kb0 == p.n_stages - 1)   // the ring is primed: ask for the tiles between it and the running prefetch
            for (int i = p.n_stages; i < min(kb1 - kb0, p.n_stages + PF_AHEAD); ++i) prefetch_b(kb0 + i, nt);
          phases ^= 1u << stage;
          if (++stage == p.n_stages) stage = 0;
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp == 1 || warp == 2) {
    // ------------------------------------------------------------------ MMA issuers (leader CTA only when paired)
    // warp 1 feeds slab 0, warp 2 slab 1: each slab has its own accumulator columns, so the two
    // instruction streams need no ordering between them; both count on the stage's `empty` barrier.
    const int sl = warp - 1;
    if (lane == 0 && leader && (sl < slabs || p.kil)) {
      const uint32_t idesc = ptx::idesc_bf16(TILE_M * CG, (uint32_t)p.tile_n);
      uint32_t phases = 0;
      int lt = 0;
      bool ok = true;
      for (int u = group; u < num_units && ok; u += n_groups, ++lt) {
        int mt, nt, kb0, kb1;
        decode(u, mt, nt, kb0, kb1);
        const int ab = lt % nbuf;
        const uint32_t aphase = (lt / nbuf) & 1;
        if (!ptx::mbar_wait(tempty_bar(ab), aphase ^ 1u)) { fail(p.status, DEV_TIMEOUT_MMA); ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (ab + sl) * ACC_COLS;   // slab sl of a two-slab unit: column sl * ACC_COLS
        int stage = 0;
        for (int kb = kb0; kb < kb1; ++kb) {
          // Alternating issuers: the ring has an even number of stages and every unit starts at stage 0, so the
          // stages of even k-blocks are the even ones.  Each stage's barriers thus have one consumer, which sees all of
          // their phases in order (a thread that skipped phases could not tell a parity from the one two phases on).
          if (p.kil && ((kb - kb0) & 1) != sl) {
            if (++stage == p.n_stages) stage = 0;
            continue;
          }
          if (!ptx::mbar_wait(full_bar(stage), (phases >> stage) & 1u)) { fail(p.status, DEV_TIMEOUT_MMA); ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint64_t a_desc = ptx::smem_desc_sw128(sA + stage * p.a_stage_bytes + (p.kil ? 0 : sl * A_STAGE_BYTES));
          const uint64_t b_desc = ptx::smem_desc_sw128(sB + stage * p.b_stage_bytes);
#pragma unroll
          for (int k = 0; k < TILE_K / 16; ++k) {   // 16 bf16 = 32 bytes per MMA: descriptor address += 2
            const uint32_t acc = (kb > kb0 + (p.kil ? sl : 0) || k > 0) ? 1u : 0u;
            if (CG == 2) ptx::mma_bf16_ss_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, acc);
            else ptx::mma_bf16_ss(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, acc);
          }
          if (CG == 2) ptx::mma_commit_pair(empty_bar(stage), 3);
          else ptx::mma_commit(empty_bar(stage));
          phases ^= 1u << stage;
          if (++stage == p.n_stages) stage = 0;
        }
        if (ok) {
          if (CG == 2) ptx::mma_commit_pair(tfull_bar(ab), 3);
          else ptx::mma_commit(tfull_bar(ab));
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp == 3 + 4 * slabs) {
    // ------------------------------------------------------------------ TMA producer of the activation tiles
    if (lane == 0) {
      const uint64_t pol_a = ptx::policy_evict_last();    // activations are re-read by every column tile
      auto issue_a = [&](int stage, int kb, int m0) {   // activation rows of k-block kb, one box per slab
        const uint32_t dstA = sA + stage * p.a_stage_bytes;
        if (CG == 1) {
          for (int sl = 0; sl < slabs; ++sl)
            ptx::tma_load_2d_hint(dstA + sl * A_STAGE_BYTES, tmA, full_bar(stage), kb * TILE_K, m0 + sl * TILE_M, pol_a);
        } else {
          const uint32_t lead_full = ptx::mapa(full_bar(stage), 0);
          for (int sl = 0; sl < slabs; ++sl)
            ptx::tma_load_2d_pair_hint(dstA + sl * A_STAGE_BYTES, tmA, lead_full, kb * TILE_K, m0 + sl * TILE_M * CG, pol_a);
        }
      };
      grid_dep_wait();   // the activations are the previous kernel's output
      uint32_t phases = 0;
      int lt = 0;
      bool ok = true;
      const bool loads_a = leader || p.a_peer_loads;   // few rows: the second CTA of a pair has none
      for (int u = group; u < num_units && ok && loads_a; u += n_groups, ++lt) {
        int mt, nt, kb0, kb1;
        decode(u, mt, nt, kb0, kb1);
        const int m0 = mt * unit_rows + (int)rank * TILE_M;
        int stage = 0;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (p.gate && lt > 0 && kb - kb0 == p.n_stages - 2 &&
              !ptx::mbar_wait(sfree_bar, (uint32_t)(lt - 1) & 1u)) { fail(p.status, DEV_TIMEOUT_PRODUCER); ok = false; break; }
          if (!ptx::mbar_wait(empty_bar(stage), ((phases >> stage) & 1u) ^ 1u)) { fail(p.status, DEV_TIMEOUT_PRODUCER); ok = false; break; }
          issue_a(stage, kb, m0);
          phases ^= 1u << stage;
          if (++stage == p.n_stages) stage = 0;
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    // warps 3-6 drain slab 0, warps 7-10 (two-slab units only) slab 1; warp w may touch TMEM lanes 32 (w % 4) ..
    const int q = warp & 3, sl = (warp - 3) >> 2;
    int lt = 0;
    bool ok = true;
    grid_dep_wait();   // the outputs may still be in use by earlier kernels until they have completed
    for (int u = group; u < num_units && ok; u += n_groups, ++lt) {
      int mt, nt, kb0, kb1;
      decode(u, mt, nt, kb0, kb1);
      const int ab = lt % nbuf;
      const uint32_t aphase = (lt / nbuf) & 1;
      if (!ptx::mbar_wait(tfull_bar(ab), aphase)) { fail(p.status, DEV_TIMEOUT_EPILOGUE); ok = false; break; }
      ptx::tc_fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (ab + sl) * ACC_COLS;
      const int row0 = mt * unit_rows + sl * (TILE_M * CG) + (int)rank * TILE_M + q * 32;
      // the staging area is idle in a CTA's last unit (every load consumed, every MMA complete, in both
      // CTAs of a pair), and in earlier units when the producer is kept off it (p.gate)
      const bool last_unit = u + n_groups >= num_units;
      const bool res_store = EPI == EPI_RESIDUAL && p.part != nullptr && p.k_splits > 1;
      const int slice_row0 = res_store ? unit_ks * p.part_rows : 0;   // partial sums: the slice's own rows
      if (EPI != EPI_LMHEAD && p.out_tma && nt < p.out_full_tiles && (last_unit || p.gate))
        drain_tile_staged<EPI>(p, tmC, taddr, slice_row0 + row0, nt, sOut + (uint32_t)(warp - 3) * (4096u * STAGE_BUFS), lane,
                               res_store);
      else
        drain_tile<EPI>(p, taddr, row0 + lane, nt, res_store ? 2 : (p.k_splits > 1 ? 1 : 0),
                        res_store ? p.part + (int64_t)slice_row0 * p.N : reinterpret_cast<float *>(p.out),
                        p.kil && kb1 - kb0 >= 2);
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        if (CG == 2) ptx::mbar_arrive_cluster(ptx::mapa(tempty_bar(ab), 0));
        else ptx::mbar_arrive(tempty_bar(ab));
        if (EPI != EPI_LMHEAD && p.gate && !last_unit) {
          ptx::bulk_wait_read();           // the TMA unit has read this warp's staging tiles
          ptx::mbar_arrive(sfree_bar);
        }
      }
    }
    if (!ok) *abort_flag = 1;
    // The TMA unit must have READ this warp's staging tiles before the CTA's shared memory goes away; the writes themselves
    // are part of the kernel's memory operations, which complete before the kernel does (and before anything ordered
    // after it, programmatic dependents included, sees its results).
    if (EPI != EPI_LMHEAD && p.out_tma && lane == 0) ptx::bulk_wait_read();
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (*abort_flag) {
    // A wait ran out: give copies still in flight time to land before the CTA's shared memory goes away.
    const uint64_t t0 = ptx::globaltimer();
    while (ptx::globaltimer() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (CG == 2) ptx::cluster_sync();     // neither CTA leaves while the other may still touch its memory
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    if (CG == 2) ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
    else ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

template <int EPI>
__global__ void __launch_bounds__(384, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmC, const KParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * MAX_STAGES + 5];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  gemm_body<EPI, 1>(&tmA, &tmB, &tmB2, &tmC, p, smem_raw, bars, &tmem_slot, &abort_flag);
}

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(384, 1)
gemm_tcgen05_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                         const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmC, const KParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * MAX_STAGES + 5];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  gemm_body<EPI, 2>(&tmA, &tmB, &tmB2, &tmC, p, smem_raw, bars, &tmem_slot, &abort_flag);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

__global__ void merge_partials_kernel(const float *part_m, const float *part_s, const int32_t *part_i,
                                      int n_tiles, int rows_padded, int32_t *pred, float *conf) {
  grid_dep_launch();
  grid_dep_wait();
  const int r = blockIdx.x, lane = threadIdx.x;
  float mx = -INFINITY, sum = 0.f;
  int ix = 0x7fffffff;
  for (int t = lane; t < n_tiles; t += 32) {
    float tm = part_m[(int64_t)t * rows_padded + r];
    float ts = part_s[(int64_t)t * rows_padded + r];
    int ti = part_i[(int64_t)t * rows_padded + r];
    if (tm > mx) { sum = sum * expf(mx - tm) + ts; mx = tm; ix = ti; }
    else { sum += ts * expf(tm - mx); if (tm == mx && ti < ix) ix = ti; }
  }
  for (int o = 16; o > 0; o >>= 1) {
    float om = __shfl_xor_sync(0xffffffffu, mx, o);
    float os = __shfl_xor_sync(0xffffffffu, sum, o);
    int oi = __shfl_xor_sync(0xffffffffu, ix, o);
    float nm = fmaxf(mx, om);
    float ns = (mx == -INFINITY ? 0.f : sum * expf(mx - nm)) + (om == -INFINITY ? 0.f : os * expf(om - nm));
    int ni = (om > mx || (om == mx && oi < ix)) ? oi : ix;
    mx = nm; sum = ns; ix = ni;
  }
  if (lane == 0) { pred[r] = ix; conf[r] = 1.0f / sum; }
}

}  // namespace

l2pd_status make_tma_2d_bf16(TmaDesc *out, const void *ptr, int64_t rows, int64_t cols, int box_rows) {
  return make_tma_2d_bf16_strided(out, ptr, rows, cols, cols, box_rows);
}

l2pd_status make_tma_2d_bf16_strided(TmaDesc *out, const void *ptr, int64_t rows, int64_t cols, int64_t row_stride,
                                     int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return L2PD_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(ptr) & 15) || (cols % 8) || (row_stride % 8) || row_stride < cols || box_rows < 1 ||
      box_rows > 256)
    return L2PD_ERR_SHAPE;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)row_stride * 2};
  cuuint32_t box[2] = {(cuuint32_t)TILE_K, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(&out->map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? L2PD_OK : L2PD_ERR_CUDA;
}

l2pd_status make_tma_out_3d(TmaDesc *out, void *ptr, bool fp32, int64_t rows, int64_t N, int tile_w) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return L2PD_ERR_CUDA;
  const int es = fp32 ? 4 : 2;
  const int64_t full = N / tile_w;
  if ((reinterpret_cast<uintptr_t>(ptr) & 15) || ((N * es) % 16) || ((tile_w * es) % 16) || full < 1 || rows < 1)
    return L2PD_ERR_SHAPE;
  cuuint64_t dims[3] = {(cuuint64_t)tile_w, (cuuint64_t)full, (cuuint64_t)rows};
  cuuint64_t strides[2] = {(cuuint64_t)tile_w * es, (cuuint64_t)N * es};
  cuuint32_t box[3] = {(cuuint32_t)(128 / es), 1, 32};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(&out->map, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, ptr, dims,
                  strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? L2PD_OK : L2PD_ERR_CUDA;
}

l2pd_status make_tma_out_tail(TmaDesc *out, void *ptr, bool fp32, int64_t rows, int64_t N, int tail_w) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return L2PD_ERR_CUDA;
  const int es = fp32 ? 4 : 2;
  if (tail_w < 1 || tail_w >= N || ((tail_w * es) % 16) || ((N * es) % 16) || rows < 1) return L2PD_ERR_SHAPE;
  uint8_t *base = reinterpret_cast<uint8_t *>(ptr) + (N - tail_w) * es;
  if (reinterpret_cast<uintptr_t>(base) & 15) return L2PD_ERR_SHAPE;
  cuuint64_t dims[3] = {(cuuint64_t)tail_w, 1, (cuuint64_t)rows};
  cuuint64_t strides[2] = {(cuuint64_t)N * es, (cuuint64_t)N * es};
  cuuint32_t box[3] = {(cuuint32_t)(128 / es), 1, 32};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(&out->map, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims,
                  strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? L2PD_OK : L2PD_ERR_CUDA;
}

// Modelled cycles of one GEMM for a tile width / K split / slab count.  Per 64-deep k-block a CTA
// needs the largest of: the tensor pipe's 2 * tile_n cycles per slab; the ~620 cycles one thread
// takes to issue its four MMAs and the stage hand-over; the bytes it must take in at INGEST bytes
// per cycle.  A unit adds a fixed fill part and, when its accumulators are not double-buffered
// (two slabs), the drain of the accumulator; times the number of waves over the SMs (or SM pairs).
static double plan_cost(int M, int N, int K, int num_sms, int cg, int slabs, int unit_n, int tile_n, int ks, bool is_residual, bool kil) {
  const double INGEST = cg == 2 ? 58.0 : 68.0;   // measured: bytes per cycle an SM takes in from L2 through TMA
  const int groups = num_sms / cg;
  const int m_tiles = ceil_div(M, TILE_M * cg * slabs);
  const int n_tiles = ceil_div(N, unit_n);
  const int units = m_tiles * n_tiles * ks;
  const int waves = ceil_div(units, groups);
  const int kb = ceil_div(ceil_div(K, TILE_K), ks);
  const double bytes = (double)slabs * A_STAGE_BYTES + 128.0 * tile_n / cg;
  const double per_kb = fmax(fmax(2.0 * tile_n * slabs, kil ? 330.0 : 620.0), bytes / INGEST) * 1.06;
  // emptying the accumulators: bf16 stores leave an SM at ~34 B per cycle; fp32 additions into X are bound
  // by L2's atomic units, ~2500 B per cycle for the whole chip, i.e. ~17 B per cycle and SM when all drain at once
  // (K slices store their partial sums plainly: twice the rate of the additions)
  const double drain = (double)TILE_M * slabs * unit_n * (is_residual ? (ks > 1 ? 4.0 / 34.0 : 4.0 / 17.0) : 2.0 / 34.0) + 1500.0;
  const double exposed = slabs == 2 ? drain : 0.3 * drain;
  return waves * (kb * per_kb + 6000.0 + exposed) + (slabs == 2 ? 0.0 : 0.7 * drain);
}

GemmPlan plan_gemm(int epi, int M, int N, int K, int num_sms, int force_tile_n, int max_k_splits, int max_tile_n) {
  GemmPlan best{1, 256, 1, 1, 0};
  double best_cost = 1e300;
  const bool swiglu = epi == EPI_SWIGLU;
  const int step = 16;   // SwiGLU: the gate and up halves are then multiples of 8 (one swizzle group of rows)
  for (int cg = 1; cg <= 2; ++cg) {
    if (cg == 2 && (M <= TILE_M || epi == EPI_LMHEAD || num_sms < 2)) continue;
    for (int slabs = 1; slabs <= 2; ++slabs) {
      // a second slab: the weight tile is read once for twice the rows, and a second thread issues MMAs
      if (slabs == 2 && (cg == 1 || epi == EPI_LMHEAD || M <= TILE_M * cg)) continue;
      for (int tn = 256; tn >= 64; tn -= step) {
        if (force_tile_n && tn != force_tile_n) continue;
        if (!force_tile_n && tn > max_tile_n) continue;
        const int unit_n = swiglu ? tn / 2 : tn;
        const int max_ks = (epi == EPI_RESIDUAL) ? (max_k_splits < 4 ? max_k_splits : 4) : 1;
        for (int ks = 1; ks <= max_ks; ++ks) {
          if (ceil_div(K, TILE_K) < 8 * ks) break;
          // few rows: one 128-row MMA per 132 cycles and issuer bounds the K loop; the idle second issuer takes every other k-block
          const bool kil = M <= TILE_M * cg && slabs == 1 && epi != EPI_LMHEAD;
          const double c = plan_cost(M, N, K, num_sms, cg, slabs, unit_n, tn, ks, epi == EPI_RESIDUAL, kil);
          if (c < best_cost - 1e-9) { best_cost = c; best = GemmPlan{cg, tn, ks, slabs, kil ? 1 : 0}; }
        }
      }
    }
  }
  if (force_tile_n && best_cost > 1e299) best.tile_n = force_tile_n;
  return best;
}

// The plan of a step of few rows inside a chained launch: SM pairs, one 256-row slab per unit, the two MMA issuers on
// alternate k-blocks; tile width and K slices by the same cost model.
GemmPlan plan_gemm_pair_one_slab(int epi, int M, int N, int K, int num_sms, int max_k_splits, int max_tile_n) {
  GemmPlan best{2, max_tile_n < 176 ? max_tile_n : 176, 1, 1, 1};
  double best_cost = 1e300;
  for (int tn = 256; tn >= 64; tn -= 16) {
    if (tn > max_tile_n) continue;
    const int unit_n = epi == EPI_SWIGLU ? tn / 2 : tn;
    const int max_ks = (epi == EPI_RESIDUAL) ? (max_k_splits < 4 ? max_k_splits : 4) : 1;
    for (int ks = 1; ks <= max_ks; ++ks) {
      if (ceil_div(K, TILE_K) < 8 * ks) break;
      const double c = plan_cost(M, N, K, num_sms, 2, 1, unit_n, tn, ks, epi == EPI_RESIDUAL, true);
      if (c < best_cost - 1e-9) { best_cost = c; best = GemmPlan{2, tn, ks, 1, 1}; }
    }
  }
  return best;
}

int lm_head_tile_n(int R, int V, int K, int num_sms) { return plan_gemm(EPI_LMHEAD, R, V, K, num_sms, 0).tile_n; }

int effective_k_splits(int K, int k_splits) {
  // every K slice must hold at least one k-block (an empty slice would add an unwritten accumulator)
  int ks = k_splits > 1 ? k_splits : 1;
  const int num_kb = ceil_div(K, TILE_K);
  while (ks > 1 && ceil_div(num_kb, ks) * (ks - 1) >= num_kb) --ks;
  return ks;
}

// Fills the kernel's parameter block for one GEMM.  stages / b_stage_bytes = 0: the deepest ring the shared
// memory holds for this tile; otherwise the given ring geometry (a kernel that runs several GEMMs keeps one ring).
cudaError_t fill_kparams(const GemmArgs &g, int stages, int b_stage_bytes, KParams &p, bool chained) {
  const int cg = g.cta_group == 2 ? 2 : 1;
  if (g.k_splits > 1 && g.epi != EPI_RESIDUAL) return cudaErrorInvalidValue;
  const int ks = effective_k_splits(g.K, g.k_splits);
  p.M = g.M; p.N = g.N; p.K = g.K; p.tile_n = g.tile_n;
  p.b_stage_bytes = b_stage_bytes > 0 ? b_stage_bytes : g.tile_n * 128 / cg;
  if (p.b_stage_bytes < g.tile_n * 128 / cg) return cudaErrorInvalidValue;
  p.slabs = g.slabs == 2 ? 2 : 1;
  if (p.slabs == 2 && g.epi == EPI_LMHEAD) return cudaErrorInvalidValue;
  p.a_stage_bytes = p.slabs * A_STAGE_BYTES;
  p.a_box_bytes = A_STAGE_BYTES;
  p.a_peer_loads = 1;
  if (g.a_box_rows > 0 && g.a_box_rows < TILE_M) {
    if (g.M > TILE_M || p.slabs != 1 || g.a_box_rows < g.M || (g.a_box_rows % 8)) return cudaErrorInvalidValue;
    p.a_box_bytes = g.a_box_rows * TILE_K * 2;
  }
  if (cg == 2 && g.M <= TILE_M) p.a_peer_loads = 0;
  const int stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
  if (stages <= 0) {
    stages = (SMEM_BUDGET - 2048) / stage_bytes;
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    if (g.k_interleave) stages &= ~1;   // alternate k-blocks <-> alternate stages
  }
  if (stages < 2 || stages > MAX_STAGES || (size_t)stages * stage_bytes + 2048 > (size_t)SMEM_BUDGET) return cudaErrorInvalidValue;
  p.n_stages = stages;
  p.m_tiles = ceil_div(g.M, TILE_M * cg * p.slabs);
  const int n_per_tile = (g.epi == EPI_SWIGLU) ? g.tile_n / 2 : g.tile_n;
  // staged output: needs the output map and a staging area (the A part of the ring's last two stages)
  p.kil = g.k_interleave ? 1 : 0;
  // single GEMM launches: alternate k-blocks <-> alternate stages (even ring), and the two-accumulator sum lives in the
  // direct-store drain; the chained kernel's issuers see every stage and its staged drain adds the accumulators
  if (p.kil && (p.slabs != 1 || g.epi == EPI_LMHEAD || (!chained && (stages & 1)))) return cudaErrorInvalidValue;
  p.out_tma = (g.c != nullptr && g.epi != EPI_LMHEAD && stages >= 3 && (!p.kil || chained)) ? 1 : 0;
  p.out_full_tiles = p.out_tma ? g.N / n_per_tile : 0;
  p.out_tail_cols = 0;
  if (p.out_tma && g.c_tail && g.tail_cols > 0) {
    if (g.tail_cols != g.N - p.out_full_tiles * n_per_tile || (g.tail_cols % (g.epi == EPI_SWIGLU ? 8 : 16))) return cudaErrorInvalidValue;
    p.out_tail_cols = g.tail_cols;
  }
  p.gate = (p.out_tma && p.slabs == 2 && stages >= 4) ? 1 : 0;
  p.n_tiles = ceil_div(g.N, n_per_tile);
  p.k_splits = ks;
  {   // a raster group's activation rows: about 32 MB, a quarter of L2
    const double tile_bytes = (double)TILE_M * cg * p.slabs * ((double)g.K / ks) * 2.0;
    int gm = (int)(32.0e6 / tile_bytes);
    p.group_m = gm < 1 ? 1 : (gm > p.m_tiles ? p.m_tiles : gm);
  }
  p.out = g.out; p.bias = g.bias; p.part_m = g.part_m; p.part_s = g.part_s; p.part_i = g.part_i;
  p.rows_padded = g.rows_padded; p.logits = g.logits; p.status = g.status;
  p.part = g.part; p.part_rows = g.part_rows;
  p.rope_cols = g.rope_cols; p.rope_dh = g.rope_dh; p.cs_stride = g.cs_stride; p.cs_table = g.cs_table; p.row_pos = g.row_pos;
  if (g.epi == EPI_QKV_ROPE && (!g.cs_table || !g.row_pos || g.rope_dh < 2 || (g.rope_dh & (g.rope_dh - 1)) || (g.rope_cols % g.rope_dh)))
    return cudaErrorInvalidValue;
  return cudaSuccess;
}

cudaError_t launch_gemm_tcgen05(cudaStream_t st, const GemmArgs &g, int num_sms) {
  const int cg = g.cta_group == 2 ? 2 : 1;
  KParams p;
  {
    cudaError_t e0 = fill_kparams(g, 0, 0, p);
    if (e0 != cudaSuccess) return e0;
  }
  const int ks = p.k_splits, stages = p.n_stages, stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
  const int units = p.m_tiles * p.n_tiles * ks;
  if (units <= 0) return cudaSuccess;
  const int groups = num_sms / cg;
  const int grid = cg * (units < groups ? units : groups);
  const size_t smem = (size_t)stages * stage_bytes + 1024;
  const CUtensorMap &b2 = g.b2 ? g.b2->map : g.b->map;
  const CUtensorMap &cm = p.out_tma ? g.c->map : g.a->map;
  cudaError_t e;
#define L2PD_LAUNCH(KERNEL, EPI)                                                                      \
  e = cudaFuncSetAttribute(KERNEL<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET - 1024); \
  if (e != cudaSuccess) return e;                                                                    \
  e = launch_kernel(KERNEL<EPI>, dim3(grid), dim3(128 + 128 * p.slabs), smem, st, g.a->map, g.b->map, b2, cm, p);                \
  if (e != cudaSuccess) return e;
  if (cg == 1) {
    switch (g.epi) {
      case EPI_STORE: L2PD_LAUNCH(gemm_tcgen05_kernel, EPI_STORE) break;
      case EPI_QKV_ROPE: L2PD_LAUNCH(gemm_tcgen05_kernel, EPI_QKV_ROPE) break;
      case EPI_RESIDUAL: L2PD_LAUNCH(gemm_tcgen05_kernel, EPI_RESIDUAL) break;
      case EPI_SWIGLU: L2PD_LAUNCH(gemm_tcgen05_kernel, EPI_SWIGLU) break;
      case EPI_LMHEAD: L2PD_LAUNCH(gemm_tcgen05_kernel, EPI_LMHEAD) break;
      default: return cudaErrorInvalidValue;
    }
  } else {
    switch (g.epi) {
      case EPI_STORE: L2PD_LAUNCH(gemm_tcgen05_pair_kernel, EPI_STORE) break;
      case EPI_QKV_ROPE: L2PD_LAUNCH(gemm_tcgen05_pair_kernel, EPI_QKV_ROPE) break;
      case EPI_RESIDUAL: L2PD_LAUNCH(gemm_tcgen05_pair_kernel, EPI_RESIDUAL) break;
      case EPI_SWIGLU: L2PD_LAUNCH(gemm_tcgen05_pair_kernel, EPI_SWIGLU) break;
      default: return cudaErrorInvalidValue;
    }
  }
#undef L2PD_LAUNCH
  return cudaGetLastError();
}

cudaError_t launch_merge_partials(cudaStream_t st, const float *part_m, const float *part_s,
                                  const int32_t *part_i, int n_tiles, int rows_padded, int R,
                                  int32_t *pred, float *conf) {
  return launch_kernel(merge_partials_kernel, dim3(R), dim3(32), 0, st, part_m, part_s, part_i, n_tiles, rows_padded, pred,
                       conf);
}

}  // namespace l2pd
