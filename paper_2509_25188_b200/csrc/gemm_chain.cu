// Several projections of a transformer layer, and the RMSNorms between them, in ONE persistent launch.
//
// At a few hundred rows every projection of the step is a single wave of tiles over the SM pairs, so a
// launch per projection exposes, each time, the launch itself, the ring fill, the accumulator drain and the
// wait for the slowest CTA.  This kernel keeps the CTAs (one pair of CTAs per SM pair, cta_group::2), their
// shared-memory ring, their barriers and their tensor memory alive over a list of phases:
//     GEMM phase   the tiles of one projection, exactly as gemm_tcgen05_pair_kernel runs them (same tiling, same
//                  epilogues, same K-slice partial sums): two 256-row slabs per unit, each with its own MMA
//                  issuer, or — for steps of at most 256 rows — one slab whose k-blocks alternate between the two
//                  issuers into two accumulators that the epilogue adds;
//     NORM phase   x += the K slices' partial sums (in slice order), n = RMSNorm(x) for the next projection.
// Between phases the CTAs meet at a counter in global memory (release add / acquire poll, bounded).  Only the
// threads that touch what another CTA wrote wait there: the producer of the activation tiles and the
// epilogue warps.  The producer of the WEIGHT tiles depends on nothing the kernel writes: it runs ahead into
// the next projection as far as the ring lets it, so the first weight tiles of a phase are already in
// shared memory (and the following ones requested into L2) when the phase opens.
//
// Warp roles: warp 0 weight producer, warps 1 and 2 MMA issuers of the two row slabs (leader CTA), warp 3
// activation producer, warps 4-11 epilogue and RMSNorm.  The first four warps are one warpgroup and the epilogue
// warps two: after set-up the first gives registers back (setmaxnreg) and the epilogue warpgroups take them, so
// that all four epilogues and the RMSNorm fit one kernel without spilling.
// Every wait is bounded; a wait that runs out sets the status word, and every role leaves its loops.
#include <math.h>

#include <new>

#include "common.cuh"
#include "gemm_device.cuh"
#include "ptx.cuh"

namespace l2pd {

using namespace gemm_dev;

namespace {

constexpr int CHAIN_MAX_PHASES = 6;
constexpr int CHAIN_MAX_GEMMS = 4;
constexpr int MAPS_PER_GEMM = 5;
constexpr int CG = 2, SLABS = 2;
constexpr int EPI_THREADS = 256;          // warps 4-11
constexpr int REGS_LAUNCH = 168, REGS_LEAN = 56, REGS_EPI = 224;   // registers per thread: at launch, producers / issuers, epilogue
static_assert(128 * REGS_LEAN + 256 * REGS_EPI <= 384 * REGS_LAUNCH, "register split exceeds what the block is launched with");
constexpr int NORM_GROUP = 128;           // threads that share one row of a NORM phase
constexpr int NORM_CACHE = 8;             // float4 per thread kept in registers between the two passes

struct NormP {
  float *x; const float *gain; bf16 *n; const float *part;
  int64_t part_stride;
  float eps;
  int rows, d, n_part;
};
struct ChainPhase {
  int is_norm, epi, map0, pad_;
  KParams g;
  NormP nm;
};
// One launch's table, in device memory (built once per row count, reused by every step): the tensor maps are read
// by the TMA unit from there, the phase records are copied to shared memory when the kernel starts.
struct alignas(128) ChainTable {
  CUtensorMap maps[CHAIN_MAX_GEMMS * MAPS_PER_GEMM];   // per GEMM phase: A, B, B2, C, C of the tail tile
  ChainPhase ph[CHAIN_MAX_PHASES];
  int n_phases, n_stages, b_stage_bytes, pad_;
  unsigned int *bar;                       // the meeting counter (monotonic)
  int32_t *status;
};
// what changes from launch to launch
struct ChainLaunch {
  const ChainTable *tab;
  unsigned int bar_base;                   // the counter's value when this launch starts
  unsigned long long *trace;               // optional [n_phases][4][gridDim.x] globaltimer stamps, see stamp()
};

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned *p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_gpu(unsigned *p, unsigned v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// orders this thread's earlier generic-proxy accesses (the acquire of the counter) before its later
// async-proxy accesses (TMA loads of what other CTAs stored), in every state space
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// One row of a NORM phase by a group of 128 threads (tid in [0, 128)): the row takes in the K slices'
// partial sums in slice order, is written back to x, and its normalised bf16 copy goes to n.
// The sum of squares is taken in the association of rmsnorm_kernel (256 threads, thread u adding elements
// u, u + 256, ... in order, warp trees, then a tree over the eight warp sums): thread t here stands in for
// that kernel's threads t (its even chunks) and t + 128 (its odd chunks), so both forms give the same bits.
template <int NPART>
__device__ __forceinline__ void norm_row(const NormP &nm, int row, int tid, int bar_id, float *red) {
  const int d = nm.d, d4 = d >> 2;
  float4 *__restrict__ xr = reinterpret_cast<float4 *>(nm.x + (int64_t)row * d);
  const float4 *__restrict__ pr = reinterpret_cast<const float4 *>(nm.part + (int64_t)row * d);
  const int64_t ps4 = nm.part_stride >> 2;
  float4 v[NORM_CACHE];
  float ss[2] = {0.f, 0.f};
  // two chunks at a time: every load of the batch is issued before the first addition or store
  constexpr int BATCH = 2;
#pragma unroll
  for (int b = 0; b < NORM_CACHE; b += BATCH) {
    float4 q[NPART > 0 ? NPART : 1][BATCH];
#pragma unroll
    for (int k = 0; k < BATCH; ++k) {
      const int i = tid + (b + k) * NORM_GROUP;
      const bool in = i < d4;
      v[b + k] = in ? xr[i] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int s = 0; s < NPART; ++s) q[s][k] = in ? pr[s * ps4 + i] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int k = 0; k < BATCH; ++k) {
      const int i = tid + (b + k) * NORM_GROUP;
      float4 &w = v[b + k];
      if (NPART > 0) {
#pragma unroll
        for (int s = 0; s < NPART; ++s) { w.x += q[s][k].x; w.y += q[s][k].y; w.z += q[s][k].z; w.w += q[s][k].w; }
        if (i < d4) xr[i] = w;
      }
      ss[(b + k) & 1] += w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
    }
  }
  for (int k = NORM_CACHE; tid + k * NORM_GROUP < d4; ++k) {   // rows longer than the register cache
    const int i = tid + k * NORM_GROUP;
    float4 w = xr[i];
    if (NPART > 0) {
#pragma unroll
      for (int s = 0; s < NPART; ++s) { const float4 q = pr[s * ps4 + i]; w.x += q.x; w.y += q.y; w.z += q.z; w.w += q.w; }
      xr[i] = w;
    }
    ss[k & 1] += w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
  }
  for (int o = 16; o > 0; o >>= 1) {
    ss[0] += __shfl_xor_sync(0xffffffffu, ss[0], o);
    ss[1] += __shfl_xor_sync(0xffffffffu, ss[1], o);
  }
  const int w4 = tid >> 5, l = tid & 31;
  named_bar_sync(bar_id, NORM_GROUP);          // the group's previous row no longer reads red
  if (l == 0) { red[w4] = ss[0]; red[4 + w4] = ss[1]; }
  named_bar_sync(bar_id, NORM_GROUP);
  float tot = (l < 8) ? red[l] : 0.f;
  for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
  const float inv = 1.0f / sqrtf(tot / (float)d + nm.eps);
  const float4 *__restrict__ g4 = reinterpret_cast<const float4 *>(nm.gain);
  bf16 *nr = nm.n + (int64_t)row * d;
  auto put = [&](int i, const float4 &w) {
    const float4 g = g4[i];
    __nv_bfloat162 lo = __floats2bfloat162_rn(w.x * g.x * inv, w.y * g.y * inv), hi = __floats2bfloat162_rn(w.z * g.z * inv, w.w * g.w * inv);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t *>(&lo);
    u.y = *reinterpret_cast<uint32_t *>(&hi);
    *reinterpret_cast<uint2 *>(nr + 4 * i) = u;
  };
#pragma unroll
  for (int k = 0; k < NORM_CACHE; ++k) {
    const int i = tid + k * NORM_GROUP;
    if (i < d4) put(i, v[k]);
  }
  for (int i = tid + NORM_CACHE * NORM_GROUP; i < d4; i += NORM_GROUP) put(i, xr[i]);   // summed and written back above, by this thread
}

// unit -> (row tile, column tile, K slice) of one GEMM phase: the order of gemm_tcgen05's kernels
__device__ __forceinline__ void decode_unit(const KParams &p, int kb_per, int num_kb, int u, int &mt, int &nt, int &ks, int &kb0,
                                            int &kb1) {
  const int per_slice = p.m_tiles * p.n_tiles;
  ks = u / per_slice;
  const int r = u - ks * per_slice;
  const int per_group = p.group_m * p.n_tiles;
  const int g = r / per_group;
  const int w = r - g * per_group;
  const int gm = min(p.group_m, p.m_tiles - g * p.group_m);
  nt = w / gm;
  mt = g * p.group_m + (w - nt * gm);
  kb0 = ks * kb_per;
  kb1 = min(num_kb, kb0 + kb_per);
}
// Bounded waits that also give up as soon as another role of this CTA has failed (abort flag) or, for the
// meeting counter, as soon as any CTA of any kernel has reported a failure (status word): one wait that runs
// out then ends the launch, and the launches queued behind it, within microseconds instead of stacking limits.
__device__ __forceinline__ bool wait_mbar(uint32_t bar, uint32_t parity, volatile int *abort_v) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = ptx::globaltimer();
  uint32_t spins = 0;
  while (!ptx::mbar_try_wait(bar, parity)) {
    if ((++spins & 0xffu) == 0) {
      if (*abort_v) return false;
      if (ptx::globaltimer() - t0 > 2000000000ull) return false;
    }
  }
  return true;
}
__device__ __forceinline__ bool wait_counter(const unsigned int *bar, unsigned target, volatile int *abort_v, const int32_t *status) {
  if ((int)(ld_acquire_gpu(bar) - target) >= 0) return true;
  const uint64_t t0 = ptx::globaltimer();
  uint32_t spins = 0;
  for (;;) {
    __nanosleep(32);
    if ((int)(ld_acquire_gpu(bar) - target) >= 0) return true;
    if ((++spins & 0x3fu) == 0) {
      if (*abort_v || (status && *reinterpret_cast<const volatile int32_t *>(status) != DEV_OK)) return false;
      if (ptx::globaltimer() - t0 > 2000000000ull) return false;
    }
  }
}

template <int NPART>
__device__ __forceinline__ void norm_row_fn(const NormP &nm, int row, int tid, int bar_id, float *red) {
  norm_row<NPART>(nm, row, tid, bar_id, red);
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(384, 1)
gemm_chain_kernel(const ChainLaunch cl) {
  const ChainTable &cp = *cl.tab;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * MAX_STAGES + 5];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int norm_go;
  __shared__ float norm_red[2][8];
  __shared__ ChainPhase s_ph[CHAIN_MAX_PHASES];   // the phase table, copied once: indexed at run time by every role

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();
  const bool leader = rank == 0;
  const int group = blockIdx.x >> 1, n_groups = gridDim.x >> 1;
  const unsigned n_ctas = gridDim.x;
  const int n_stages = cp.n_stages, b_stage_bytes = cp.b_stage_bytes;
  const int a_stage_bytes = SLABS * A_STAGE_BYTES;
  unsigned int *const g_bar = cp.bar;
  int32_t *const g_status = cp.status;

  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = base;
  const uint32_t sB = base + n_stages * a_stage_bytes;
  const uint32_t sOut = sA + (uint32_t)(n_stages - 2) * a_stage_bytes;   // output staging over the A part of the last two stages
  const uint32_t bar0 = ptx::smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (MAX_STAGES + s); };
  const uint32_t tfull_bar = bar0 + 8u * (2 * MAX_STAGES);
  const uint32_t tempty_bar = bar0 + 8u * (2 * MAX_STAGES + 2);
  const uint32_t sfree_bar = bar0 + 8u * (2 * MAX_STAGES + 4);

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) { ptx::mbar_init(full_bar(s), 1); ptx::mbar_init(empty_bar(s), SLABS); }
    ptx::mbar_init(tfull_bar, SLABS);
    ptx::mbar_init(tempty_bar, 4 * CG * SLABS);
    ptx::mbar_init(sfree_bar, 4 * SLABS);
    abort_flag = 0;
    norm_go = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  {
    static_assert(sizeof(ChainPhase) % 4 == 0, "phase record");
    const uint32_t *src = reinterpret_cast<const uint32_t *>(cp.ph);
    uint32_t *dst = reinterpret_cast<uint32_t *>(s_ph);
    for (int i = threadIdx.x; i < (int)(sizeof(ChainPhase) * CHAIN_MAX_PHASES / 4); i += blockDim.x) dst[i] = __ldg(src + i);
  }
  if (warp == 0 && lane < CHAIN_MAX_GEMMS * MAPS_PER_GEMM) ptx::prefetch_tensormap(&cp.maps[lane]);
  const int n_phases = cp.n_phases;
  if (warp == 1) { ptx::tmem_alloc_pair(ptx::smem_u32(&tmem_slot), TMEM_COLS); ptx::tmem_relinquish_pair(); }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::cluster_sync();     // the peer's barriers exist before anything arrives on them
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = tmem_slot;
  grid_dep_launch();

  // the counter's value once every CTA has finished phase ph
  auto bar_target = [&](int ph) { return cl.bar_base + (unsigned)(ph + 1) * n_ctas; };
  // trace stamps of a phase, per CTA: 0 opened (the phase before is complete everywhere), 1 the CTA's first accumulator
  // is ready, 2 its last accumulator is ready, 3 finished (outputs stored)
  auto stamp = [&](int ph, int what) {
    if (cl.trace) cl.trace[((int64_t)ph * 4 + what) * n_ctas + blockIdx.x] = ptx::globaltimer();
  };
  volatile int *abort_v = &abort_flag;
  auto wait_bar = [&](uint32_t bar, uint32_t parity) -> bool { return wait_mbar(bar, parity, abort_v); };
  auto wait_grid = [&](unsigned target) -> bool { return wait_counter(g_bar, target, abort_v, g_status); };

  // 384 threads x REGS_LAUNCH registers at launch = 128 x REGS_LEAN + 256 x REGS_EPI
  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_LEAN));
  if (warp == 0) {
    // ------------------------------------------------------------------ weight producer (runs ahead through the phases)
    if (lane == 0) {
      const uint64_t pol_w = ptx::policy_evict_first();
      uint32_t phases = 0;
      bool ok = true;
      constexpr int PF_AHEAD = 8;
      for (int ph = 0; ph < n_phases && ok; ++ph) {
        if (s_ph[ph].is_norm) continue;
        const KParams &p = s_ph[ph].g;
        const int epi = s_ph[ph].epi;
        const CUtensorMap *tmB = &cp.maps[s_ph[ph].map0 + 1], *tmB2 = &cp.maps[s_ph[ph].map0 + 2];
        const int half_n = p.tile_n >> 1;
        const uint32_t tx = (1 + p.a_peer_loads) * (uint32_t)p.slabs * p.a_box_bytes + CG * (uint32_t)half_n * 128u;
        const int num_units = p.m_tiles * p.n_tiles * p.k_splits;
        const int num_kb = (p.K + TILE_K - 1) / TILE_K, kb_per = (num_kb + p.k_splits - 1) / p.k_splits;
        const CUtensorMap *mine = (epi == EPI_SWIGLU) ? (leader ? tmB : tmB2) : tmB;
        for (int u = group; u < num_units && ok; u += n_groups) {
          int mt, nt, ks, kb0, kb1;
          decode_unit(p, kb_per, num_kb, u, mt, nt, ks, kb0, kb1);
          const int brow = (epi == EPI_SWIGLU) ? nt * half_n : nt * p.tile_n + (int)rank * half_n;
          int stage = 0;
          for (int kb = kb0; kb < kb1; ++kb) {
            if (kb + n_stages + PF_AHEAD < kb1) ptx::tma_prefetch_l2_2d(mine, (kb + n_stages + PF_AHEAD) * TILE_K, brow);
            if (!wait_bar(empty_bar(stage), ((phases >> stage) & 1u) ^ 1u)) { fail(g_status, DEV_TIMEOUT_PRODUCER); ok = false; break; }
            if (leader) ptx::mbar_arrive_expect_tx(full_bar(stage), tx);
            ptx::tma_load_2d_pair_hint(sB + stage * b_stage_bytes, mine, ptx::mapa(full_bar(stage), 0), kb * TILE_K, brow, pol_w);
            if (kb - kb0 == n_stages - 1)   // the ring is primed: ask for the tiles between it and the running prefetch
              for (int i = n_stages; i < min(kb1 - kb0, n_stages + PF_AHEAD); ++i) ptx::tma_prefetch_l2_2d(mine, (kb0 + i) * TILE_K, brow);
            phases ^= 1u << stage;
            if (++stage == n_stages) stage = 0;
          }
        }
      }
      if (!ok) abort_flag = 1;
    }
  } else if (warp == 1 || warp == 2) {
    // ------------------------------------------------------------------ MMA issuers (leader CTA)
    // Two slabs: warp 1 feeds slab 0, warp 2 slab 1 (separate accumulators, no ordering between the two streams).
    // One slab: the two issuers take alternate k-blocks of the unit into two accumulators (an issuer is limited to
    // one instruction per ~132 cycles, which alone would bound a K loop of few rows).  Either way BOTH issuers wait
    // on every stage's `full` barrier and commit once on its `empty` barrier, so every barrier sees the same two
    // arrivals per use whatever the phase's shape, and no issuer ever skips a barrier phase.
    const int sl = warp - 1;
    if (lane == 0 && leader) {
      uint32_t phases = 0;
      int lt = 0;
      bool ok = true;
      const uint32_t d_tmem = tmem_base + sl * ACC_COLS;
      for (int ph = 0; ph < n_phases && ok; ++ph) {
        if (s_ph[ph].is_norm) continue;
        const KParams &p = s_ph[ph].g;
        const uint32_t idesc = ptx::idesc_bf16(TILE_M * CG, (uint32_t)p.tile_n);
        const int num_units = p.m_tiles * p.n_tiles * p.k_splits;
        const int num_kb = (p.K + TILE_K - 1) / TILE_K, kb_per = (num_kb + p.k_splits - 1) / p.k_splits;
        const bool alternate = p.slabs == 1;
        for (int u = group; u < num_units && ok; u += n_groups, ++lt) {
          int mt, nt, ks, kb0, kb1;
          decode_unit(p, kb_per, num_kb, u, mt, nt, ks, kb0, kb1);
          if (!wait_bar(tempty_bar, ((uint32_t)lt & 1u) ^ 1u)) { fail(g_status, DEV_TIMEOUT_MMA); ok = false; break; }
          ptx::tc_fence_after_sync();
          int stage = 0;
          for (int kb = kb0; kb < kb1; ++kb) {
            if (!wait_bar(full_bar(stage), (phases >> stage) & 1u)) { fail(g_status, DEV_TIMEOUT_MMA); ok = false; break; }
            ptx::tc_fence_after_sync();
            if (!alternate || ((kb - kb0) & 1) == sl) {
              const uint64_t a_desc = ptx::smem_desc_sw128(sA + stage * a_stage_bytes + (alternate ? 0 : sl * A_STAGE_BYTES));
              const uint64_t b_desc = ptx::smem_desc_sw128(sB + stage * b_stage_bytes);
              const int first_kb = kb0 + (alternate ? sl : 0);       // this accumulator's first k-block
#pragma unroll
              for (int k = 0; k < TILE_K / 16; ++k)
                ptx::mma_bf16_ss_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb > first_kb || k > 0) ? 1u : 0u);
            }
            ptx::mma_commit_pair(empty_bar(stage), 3);
            phases ^= 1u << stage;
            if (++stage == n_stages) stage = 0;
          }
          if (ok) ptx::mma_commit_pair(tfull_bar, 3);
        }
      }
      if (!ok) abort_flag = 1;
    }
  } else if (warp == 3) {
    // ------------------------------------------------------------------ activation producer
    if (lane == 0) {
      const uint64_t pol_a = ptx::policy_evict_last();
      grid_dep_wait();   // phase 0 reads what the previous kernel of the stream wrote
      uint32_t phases = 0;
      int lt = 0;
      // an earlier launch of the stream has failed: its outputs are not there, do nothing (the host reports it)
      bool ok = !(g_status && *reinterpret_cast<volatile int32_t *>(g_status) != DEV_OK);
      for (int ph = 0; ph < n_phases && ok; ++ph) {
        if (s_ph[ph].is_norm) continue;
        const KParams &p = s_ph[ph].g;
        const CUtensorMap *tmA = &cp.maps[s_ph[ph].map0];
        const int num_units = p.m_tiles * p.n_tiles * p.k_splits;
        const int num_kb = (p.K + TILE_K - 1) / TILE_K, kb_per = (num_kb + p.k_splits - 1) / p.k_splits;
        if (ph > 0) {   // this phase's activations: written by every CTA during the phase before
          if (!wait_grid(bar_target(ph - 1))) { fail(g_status, DEV_TIMEOUT_PRODUCER); ok = false; break; }
          fence_proxy_async_all();
        }
        const bool loads_a = leader || p.a_peer_loads;   // few rows: the second CTA of a pair has none
        for (int u = group; u < num_units && ok && loads_a; u += n_groups, ++lt) {
          int mt, nt, ks, kb0, kb1;
          decode_unit(p, kb_per, num_kb, u, mt, nt, ks, kb0, kb1);
          const int m0 = mt * (TILE_M * CG * p.slabs) + (int)rank * TILE_M;
          int stage = 0;
          for (int kb = kb0; kb < kb1; ++kb) {
            // the last two stages' A parts double as the epilogue's staging area: refill them only once the
            // unit before has handed its output to the TMA unit
            if (lt > 0 && kb - kb0 == n_stages - 2 && !wait_bar(sfree_bar, (uint32_t)(lt - 1) & 1u)) { fail(g_status, DEV_TIMEOUT_PRODUCER); ok = false; break; }
            if (!wait_bar(empty_bar(stage), ((phases >> stage) & 1u) ^ 1u)) { fail(g_status, DEV_TIMEOUT_PRODUCER); ok = false; break; }
            const uint32_t dstA = sA + stage * a_stage_bytes;
            const uint32_t lead_full = ptx::mapa(full_bar(stage), 0);
            for (int sl = 0; sl < p.slabs; ++sl)
              ptx::tma_load_2d_pair_hint(dstA + sl * A_STAGE_BYTES, tmA, lead_full, kb * TILE_K, m0 + sl * TILE_M * CG, pol_a);
            phases ^= 1u << stage;
            if (++stage == n_stages) stage = 0;
          }
        }
      }
      if (!ok) abort_flag = 1;
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_EPI));
    // ------------------------------------------------------------------ epilogue warps 4-11: drain, RMSNorm, phase hand-over
    const int q = warp & 3, sl = (warp - 4) >> 2;
    const int etid = threadIdx.x - 128;   // 0 .. 255
    int lt = 0;
    grid_dep_wait();   // the outputs may still be in use by earlier kernels until they have completed
    bool ok = !(g_status && *reinterpret_cast<volatile int32_t *>(g_status) != DEV_OK);
    if (!ok) abort_flag = 1;
    for (int ph = 0; ph < n_phases; ++ph) {
      const ChainPhase &P = s_ph[ph];
      if (!P.is_norm) {
        // by value: the fields the epilogue uses live in registers for the phase (read through a pointer to shared
        // memory they would be re-read after every tensor-memory instruction)
        const KParams p = P.g;
        const CUtensorMap *tmC = &cp.maps[P.map0 + 3];   // tmC + 1: the tail tile's map
        const int num_units = p.m_tiles * p.n_tiles * p.k_splits;
        const int num_kb = (p.K + TILE_K - 1) / TILE_K, kb_per = (num_kb + p.k_splits - 1) / p.k_splits;
        if (ph > 0 && ok && group < num_units) {   // order this warp's global accesses after the phase before
          int w = 1;
          if (lane == 0) w = wait_grid(bar_target(ph - 1)) ? 1 : 0;
          w = __shfl_sync(0xffffffffu, w, 0);
          if (!w) { fail(g_status, DEV_TIMEOUT_EPILOGUE); ok = false; }
        }
        if (etid == 0) { stamp(ph, 0); stamp(ph, 1); stamp(ph, 2); }
        for (int u = group; u < num_units && ok; u += n_groups, ++lt) {
          int mt, nt, ks, kb0, kb1;
          decode_unit(p, kb_per, num_kb, u, mt, nt, ks, kb0, kb1);
          const int row0 = mt * (TILE_M * CG * p.slabs) + sl * (TILE_M * CG) + (int)rank * TILE_M + q * 32;
          if (!wait_bar(tfull_bar, (uint32_t)lt & 1u)) { fail(g_status, DEV_TIMEOUT_EPILOGUE); ok = false; break; }
          ptx::tc_fence_after_sync();
          if (etid == 0) { if (u == group) stamp(ph, 1); stamp(ph, 2); }
          const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (p.slabs == 2 ? sl * ACC_COLS : 0);
          const bool res_store = P.epi == EPI_RESIDUAL && p.part != nullptr && p.k_splits > 1;
          const int slice_row0 = res_store ? ks * p.part_rows : 0;
          const uint32_t stage0 = sOut + (uint32_t)(warp - 4) * (4096u * STAGE_BUFS);
          // every tile goes through the staging area and the TMA unit; the row's last, narrower tile has a map of its own.
          // One-slab phases: the second group of epilogue warps has no rows (it only takes part in the hand-overs below),
          // and the unit's sum is the two issuers' accumulators added.
          const int tail = nt < p.out_full_tiles ? 0 : p.out_tail_cols;
          const CUtensorMap *tm = tail ? tmC + 1 : tmC;
          const bool two_acc = p.slabs == 1;
          if (sl < p.slabs) {
            switch (P.epi) {
              case EPI_QKV_ROPE: drain_tile_staged<EPI_QKV_ROPE>(p, tm, taddr, slice_row0 + row0, nt, stage0, lane, res_store, tail); break;
              case EPI_RESIDUAL: drain_tile_staged<EPI_RESIDUAL>(p, tm, taddr, slice_row0 + row0, nt, stage0, lane, res_store, tail, two_acc); break;
              case EPI_SWIGLU: drain_tile_staged<EPI_SWIGLU>(p, tm, taddr, slice_row0 + row0, nt, stage0, lane, res_store, tail, two_acc); break;
              default: drain_tile_staged<EPI_STORE>(p, tm, taddr, slice_row0 + row0, nt, stage0, lane, res_store, tail, two_acc); break;
            }
          }
          ptx::tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            ptx::mbar_arrive_cluster(ptx::mapa(tempty_bar, 0));
            ptx::bulk_wait_read();           // the TMA unit has read this warp's staging tiles
            ptx::mbar_arrive(sfree_bar);
          }
        }
        if (lane == 0) ptx::bulk_wait_all();   // this warp's staged stores have reached memory
        __threadfence();
      } else {
        // RMSNorm phase: two rows at a time per CTA, 128 threads each
        if (etid == 0) {
          int go = (abort_flag == 0 && ok) ? 1 : 0;
          if (go && ph > 0 && !wait_grid(bar_target(ph - 1))) { fail(g_status, DEV_TIMEOUT_EPILOGUE); go = 0; abort_flag = 1; }
          norm_go = go;
          stamp(ph, 0); stamp(ph, 1); stamp(ph, 2);
        }
        __syncwarp();
        named_bar_sync(1, EPI_THREADS);
        const bool go = norm_go != 0;
        if (go) {
          const NormP &nm = P.nm;
          const int g2 = etid / NORM_GROUP, tid = etid - g2 * NORM_GROUP;
          for (int row = 2 * (int)blockIdx.x + g2; row < nm.rows; row += 2 * (int)n_ctas) {
            switch (nm.n_part) {
              case 0: norm_row_fn<0>(nm, row, tid, 2 + g2, norm_red[g2]); break;
              case 2: norm_row_fn<2>(nm, row, tid, 2 + g2, norm_red[g2]); break;
              case 3: norm_row_fn<3>(nm, row, tid, 2 + g2, norm_red[g2]); break;
              default: norm_row_fn<4>(nm, row, tid, 2 + g2, norm_red[g2]); break;
            }
          }
        } else {
          ok = false;
        }
        __threadfence();
      }
      // phase hand-over: all eight warps of this CTA are done with the phase -> one arrival on the counter
      __syncwarp();
      named_bar_sync(1, EPI_THREADS);
      if (etid == 0) {
        stamp(ph, 3);
        if (ph + 1 < n_phases) {
          fence_proxy_async_all();
          __threadfence();
          red_release_gpu(g_bar, 1u);
        }
      }
    }
    if (!ok) abort_flag = 1;
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
  ptx::cluster_sync();     // neither CTA leaves while the other may still touch its memory
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

}  // namespace

int chain_max_clusters(int num_sms) {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (cached[dev]) return cached[dev] > 0 ? cached[dev] : 0;
  int n = 0;
  if (cudaFuncSetAttribute(gemm_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET - 4096 + 1024) == cudaSuccess) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(num_sms & ~1);
    cfg.blockDim = dim3(384);
    cfg.dynamicSmemBytes = SMEM_BUDGET - 4096 + 1024;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_chain_kernel, &cfg) != cudaSuccess) { n = 0; cudaGetLastError(); }
  }
  if (n > num_sms / 2) n = num_sms / 2;
  cached[dev] = n > 0 ? n : -1;
  return n > 0 ? n : 0;
}

bool chain_step_supported(const ChainStep &s) {
  if (s.is_norm) return s.nm.d % 4 == 0 && (s.nm.n_part == 0 || (s.nm.n_part >= 2 && s.nm.n_part <= 4));
  const GemmArgs &g = s.g;
  // SM pairs; two slabs with an issuer each, or one slab with the two issuers on alternate k-blocks
  if (g.cta_group != 2) return false;
  if (!((g.slabs == 2 && !g.k_interleave) || (g.slabs <= 1 && g.k_interleave))) return false;
  if (g.epi != EPI_STORE && g.epi != EPI_QKV_ROPE && g.epi != EPI_RESIDUAL && g.epi != EPI_SWIGLU) return false;
  if (g.epi == EPI_QKV_ROPE && g.slabs != 2) return false;   // the rotating epilogue does not add two accumulators
  if (g.tile_n < 32 || g.tile_n > 256 || (g.tile_n % 16)) return false;
  // a K split must leave every unit at least a ring's worth of k-blocks (the staging gate is taken once per unit)
  const int ks = effective_k_splits(g.K, g.k_splits);
  const int num_kb = ceil_div(g.K, TILE_K);
  if (ceil_div(num_kb, ks) * (ks - 1) >= num_kb) return false;
  if (num_kb - ceil_div(num_kb, ks) * (ks - 1) < MAX_STAGES) return false;
  if (g.epi == EPI_RESIDUAL && ks > 1 && !g.part) return false;   // K slices must store partial sums (fixed order)
  // every tile is stored through the TMA unit: an output map, and one for the last tile if it is narrower
  const int n_per_tile = g.epi == EPI_SWIGLU ? g.tile_n / 2 : g.tile_n;
  if (!g.c || g.N < n_per_tile) return false;
  const int tail = g.N % n_per_tile;
  if (tail && (!g.c_tail || g.tail_cols != tail || (tail % (g.epi == EPI_SWIGLU ? 8 : 16)))) return false;
  return true;
}

size_t chain_table_bytes() { return sizeof(ChainTable); }

cudaError_t chain_build_table(const ChainStep *steps, int n_steps, unsigned int *bar, int32_t *status, void *h_table,
                              ChainTableInfo *info) {
  if (n_steps < 1 || n_steps > CHAIN_MAX_PHASES || !bar || !status || !h_table || !info) return cudaErrorInvalidValue;
  ChainTable &c = *new (h_table) ChainTable();
  int max_b = 0, n_gemm = 0;
  for (int i = 0; i < n_steps; ++i) {
    if (!chain_step_supported(steps[i])) return cudaErrorInvalidValue;
    if (steps[i].is_norm) continue;
    if (++n_gemm > CHAIN_MAX_GEMMS) return cudaErrorInvalidValue;
    const int b = steps[i].g.tile_n * 128 / CG;
    if (b > max_b) max_b = b;
  }
  if (steps[0].is_norm) return cudaErrorInvalidValue;   // the first phase orders the launch after the stream's previous kernel
  max_b = (max_b + 1023) & ~1023;
  const int stage_bytes = SLABS * A_STAGE_BYTES + max_b;
  int stages = (SMEM_BUDGET - 4096) / stage_bytes;   // the kernel's static shared memory (phase table, barriers) is ~2 KB
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages < 4) return cudaErrorInvalidValue;   // two stages double as the staging area
  c.n_phases = n_steps; c.n_stages = stages; c.b_stage_bytes = max_b; c.pad_ = 0;
  c.bar = bar; c.status = status;
  int mi = 0;
  for (int i = 0; i < n_steps; ++i) {
    ChainPhase &P = c.ph[i];
    P.is_norm = steps[i].is_norm ? 1 : 0;
    P.epi = 0; P.map0 = 0; P.pad_ = 0;
    if (steps[i].is_norm) {
      const ChainNorm &nm = steps[i].nm;
      if (nm.n_part > 0 && (nm.part_stride % 4)) return cudaErrorInvalidValue;
      P.nm.x = nm.x; P.nm.gain = nm.gain; P.nm.n = nm.n; P.nm.part = nm.part; P.nm.part_stride = nm.part_stride;
      P.nm.eps = nm.eps; P.nm.rows = nm.rows; P.nm.d = nm.d; P.nm.n_part = nm.n_part;
      continue;
    }
    const GemmArgs &g = steps[i].g;
    cudaError_t e = fill_kparams(g, stages, max_b, P.g, true);
    if (e != cudaSuccess) return e;
    P.g.status = status;
    P.epi = g.epi;
    if (!P.g.out_tma || (g.N % (g.epi == EPI_SWIGLU ? g.tile_n / 2 : g.tile_n) != 0 && !P.g.out_tail_cols)) return cudaErrorInvalidValue;
    P.map0 = MAPS_PER_GEMM * mi;
    c.maps[P.map0 + 0] = g.a->map;
    c.maps[P.map0 + 1] = g.b->map;
    c.maps[P.map0 + 2] = g.b2 ? g.b2->map : g.b->map;
    c.maps[P.map0 + 3] = g.c->map;
    c.maps[P.map0 + 4] = P.g.out_tail_cols ? g.c_tail->map : g.c->map;
    ++mi;
  }
  for (; mi < CHAIN_MAX_GEMMS; ++mi)
    for (int k = 0; k < MAPS_PER_GEMM; ++k) c.maps[MAPS_PER_GEMM * mi + k] = c.maps[0];   // every slot holds a valid map (all are prefetched)
  info->n_phases = n_steps;
  info->n_stages = stages;
  info->smem_bytes = (size_t)stages * stage_bytes + 1024;
  return cudaSuccess;
}

cudaError_t launch_gemm_chain(cudaStream_t st, const void *d_table, const ChainTableInfo &info, int n_clusters,
                              unsigned int *bar_base, unsigned long long *trace) {
  if (!d_table || n_clusters < 1 || !bar_base || info.n_phases < 1) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(gemm_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET - 4096 + 1024);
  if (e != cudaSuccess) return e;
  ChainLaunch cl;
  cl.tab = reinterpret_cast<const ChainTable *>(d_table);
  cl.bar_base = *bar_base;
  cl.trace = trace;
  e = launch_kernel(gemm_chain_kernel, dim3(2 * n_clusters), dim3(384), info.smem_bytes, st, cl);
  if (e != cudaSuccess) return e;
  *bar_base += (unsigned)(info.n_phases - 1) * (unsigned)(2 * n_clusters);
  return cudaGetLastError();
}

}  // namespace l2pd
