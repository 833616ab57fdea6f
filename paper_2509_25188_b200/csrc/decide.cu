// Decision kernel: everything of a denoising step that follows M(X).
//   * merges the LM head's per-vocabulary-tile (max, sum-exp, argmax) records into the greedy
//     prediction (Eq. 3) and its confidence (Eq. 4);
//   * runs the filter f_theta on the block's s confidences, z = W2 relu(W1 c + b1) + b2,
//     p = sigmoid(z) (Section 3.2);
//   * Algorithm 2: every masked position with p > tau (strict) is committed in place; if none
//     passes, the masked position with the highest confidence is committed so the loop advances;
//     (comparison policies of Section 3.1 replace the test: confidence above a fixed threshold, or
//     Extremely Greedy Parallel, prediction == reference token; an EGP step in which nothing
//     matches commits the reference token at the most confident masked position);
//   * EoTP (Section 3.3): the earliest committed [EoT] cuts the sequence; later positions leave
//     the mask set and read as [EoT];
//   * block advance / stop (Algorithm 3: no block after one that holds [EoT]).
// One thread block per sequence taking part in the step (a warp per block row where possible).
#include "common.cuh"

namespace l2pd {

namespace {

constexpr int MAX_S = 64;

__global__ void __launch_bounds__(1024) decide_kernel(DecideArgs a) {
  __shared__ float s_conf[MAX_S];
  __shared__ int s_pred[MAX_S];
  __shared__ float s_c[MAX_S];
  __shared__ float s_h[MAX_S];
  __shared__ float s_t[MAX_S];
  __shared__ float s_p[MAX_S];
  __shared__ int s_masked[MAX_S];
  __shared__ int s_unmask[MAX_S];
  __shared__ int s_commit[MAX_S];
  __shared__ int s_any, s_forced, s_e, s_left;

  grid_dep_launch();
  grid_dep_wait();
  const int slot = blockIdx.x;
  const SeqMeta m = a.meta[slot];
  const int s = a.s;
  const int seq = m.seq;
  const int g0 = m.block * s;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;

  // ---- confidence head: merge tile records, row r = slot*s + j -------------------------------
  for (int j = warp; j < s; j += n_warps) {
    float mx = -INFINITY, sum = 0.f;
    int ix = 0x7fffffff;
    if (j < m.n_blk_rows) {
      int r = slot * s + j;
      // eight records per lane are requested before the first is folded in (the fold order is unchanged)
      constexpr int U = 8;
      for (int t0 = lane; t0 < a.n_tiles; t0 += 32 * U) {
        float tm[U], ts[U];
        int ti[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int t = t0 + 32 * u;
          const bool in = t < a.n_tiles;
          const int64_t o = (int64_t)(in ? t : t0) * a.rows_padded + r;
          tm[u] = in ? a.part_m[o] : -INFINITY;
          ts[u] = in ? a.part_s[o] : 0.f;
          ti[u] = in ? a.part_i[o] : 0x7fffffff;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          if (t0 + 32 * u >= a.n_tiles) break;
          if (tm[u] > mx) { sum = sum * expf(mx - tm[u]) + ts[u]; mx = tm[u]; ix = ti[u]; }
          else { sum += ts[u] * expf(tm[u] - mx); if (tm[u] == mx && ti[u] < ix) ix = ti[u]; }
        }
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
    }
    if (lane == 0) {
      bool live = j < m.n_blk_rows;
      s_conf[j] = live ? 1.0f / sum : 0.f;
      s_pred[j] = live ? ix : -1;
    }
  }
  if (threadIdx.x < s) {
    int j = threadIdx.x;
    s_masked[j] = a.masked[(int64_t)seq * a.G + g0 + j];
    s_unmask[j] = 0;
  }
  if (threadIdx.x == 0) { s_any = 0; s_forced = 0; s_e = 0x7fffffff; s_left = 0; }
  __syncthreads();

  // ---- filter ----------------------------------------------------------------------------------
  if (threadIdx.x < s) {
    int j = threadIdx.x;
    float c = (j < m.n_blk_rows) ? s_conf[j] : 1.0f;       // positions cut off by EoTP read as finished
    if (a.committed_conf_mode == 1 && !s_masked[j]) c = 1.0f;
    s_c[j] = c;
  }
  __syncthreads();
  if (a.use_filter && a.rule == 0 && a.n_filter_layers > 0) {
    // depth variants: x <- W_k x + b_k with ReLU between consecutive layers; s_h / s_t alternate as output
    // (s_c, the filter's input, stays intact for the sample sink)
    float *src = s_c, *dst = s_h;
    for (int k = 0; k < a.n_filter_layers; ++k) {
      if (threadIdx.x < s) {
        const int j = threadIdx.x;
        float z = a.fb[k][j];
        for (int i = 0; i < s; ++i) z = fmaf(a.fw[k][j * s + i], k > 0 ? fmaxf(src[i], 0.f) : src[i], z);
        dst[j] = z;
        if (k + 1 == a.n_filter_layers) s_p[j] = 1.0f / (1.0f + expf(-z));
      }
      __syncthreads();
      src = dst; dst = (dst == s_h) ? s_t : s_h;
    }
  } else if (a.use_filter && a.rule == 0) {
    if (threadIdx.x < s) {
      int j = threadIdx.x;
      float h = a.b1[j];
      for (int i = 0; i < s; ++i) h = fmaf(a.w1[j * s + i], s_c[i], h);
      s_h[j] = fmaxf(h, 0.f);
    }
    __syncthreads();
    if (threadIdx.x < s) {
      int j = threadIdx.x;
      float z = a.b2[j];
      for (int i = 0; i < s; ++i) z = fmaf(a.w2[j * s + i], s_h[i], z);
      s_p[j] = 1.0f / (1.0f + expf(-z));
    }
  } else if (threadIdx.x < s) {
    s_p[threadIdx.x] = 0.f;
  }
  __syncthreads();

  // ---- threshold, progress fallback ------------------------------------------------------------------
  if (threadIdx.x < s) {
    int j = threadIdx.x;
    bool pass;
    if (a.rule == 0) pass = s_p[j] > a.tau;
    else if (a.rule == 1) pass = s_conf[j] > a.conf_threshold;
    else pass = s_pred[j] == a.ref[(int64_t)seq * a.G + g0 + j];   // dead rows hold -1, never a token id
    s_commit[j] = s_pred[j];
    if (s_masked[j] && pass) { s_unmask[j] = 1; s_any = 1; }
  }
  __syncthreads();
  // Nothing passed: thread 0 commits the most confident masked position.  s_any is not written after the barrier
  // above, and every thread takes the barrier below, so all warps run the same number of barriers whatever they read.
  if (threadIdx.x == 0 && s_any == 0) {
    int best = -1;
    float bc = -1.f;
    for (int j = 0; j < s; ++j)
      if (s_masked[j] && s_conf[j] > bc) { bc = s_conf[j]; best = j; }
    if (best >= 0) {
      s_unmask[best] = 1; s_forced = 1;
      if (a.rule == 2) s_commit[best] = a.ref[(int64_t)seq * a.G + g0 + best];
    }
  }
  __syncthreads();
  const int forced = s_forced;

  // ---- commit in place ----------------------------------------------------------------------------
  if (threadIdx.x < s) {
    int j = threadIdx.x;
    if (s_unmask[j]) {
      a.tokens[(int64_t)seq * a.tok_stride + m.blk_start + j] = s_commit[j];
      a.masked[(int64_t)seq * a.G + g0 + j] = 0;
      s_masked[j] = 0;
      if (a.use_eotp && s_commit[j] == a.eot_id) atomicMin(&s_e, g0 + j);
    }
    if (a.collect_c) {   // stage 1 of Algorithm 1: the filter's input and the target y_j = [pred_j == r_j]
      const int64_t row = a.collect_base + slot;
      a.collect_c[row * s + j] = s_c[j];
      a.collect_y[row * s + j] = (a.rule == 2 && s_pred[j] == a.ref[(int64_t)seq * a.G + g0 + j]) ? 1 : 0;
    }
    if (a.o_conf) a.o_conf[(int64_t)seq * s + j] = s_conf[j];
    if (a.o_pred) a.o_pred[(int64_t)seq * s + j] = s_pred[j];
    if (a.o_p) a.o_p[(int64_t)seq * s + j] = s_p[j];
    if (a.o_unmask) a.o_unmask[(int64_t)seq * s + j] = (uint8_t)s_unmask[j];
  }
  __syncthreads();

  // ---- EoTP -------------------------------------------------------------------------------------
  int e = a.st.eot_pos[seq];
  int l_eff = a.st.l_eff[seq];
  if (a.use_eotp && s_e != 0x7fffffff && (e < 0 || s_e < e)) {
    e = s_e;
    l_eff = a.P + e + 1;
    for (int g = e + 1 + threadIdx.x; g < a.G; g += blockDim.x) {
      a.masked[(int64_t)seq * a.G + g] = 0;
      a.tokens[(int64_t)seq * a.tok_stride + a.P + g] = a.eot_id;
    }
    if (threadIdx.x < s && g0 + threadIdx.x > e) s_masked[threadIdx.x] = 0;
  }
  __syncthreads();
  if (threadIdx.x < s && s_masked[threadIdx.x]) atomicAdd(&s_left, 1);
  __syncthreads();

  // ---- block advance / stop -------------------------------------------------------------------------
  if (threadIdx.x == 0) {
    int cur = m.block, done = 0;
    if (s_left == 0) {
      if (e >= 0 || cur + 1 == a.n_blocks) done = 1;
      else cur += 1;
    }
    a.st.cur_block[seq] = cur;
    a.st.l_eff[seq] = l_eff;
    a.st.eot_pos[seq] = e;
    a.st.done[seq] = done;
    a.st.steps[seq] += 1;
    a.st.forced[seq] += forced;
    StepSummary sm;
    sm.block = m.block; sm.masks_left = s_left; sm.l_eff = l_eff; sm.done = done;
    sm.forced = forced; sm.cur_block = cur;
    a.summary[seq] = sm;
  }
}

}  // namespace

cudaError_t launch_decide(cudaStream_t st, const DecideArgs &a, int n_slots) {
  // one warp per block row for the merge of the tile records (the latency-bound part): up to 32 warps
  int threads = 32 * a.s;
  threads = threads < 256 ? 256 : (threads > 1024 ? 1024 : threads);
  return launch_kernel(decide_kernel, dim3(n_slots), dim3(threads), 0, st, a);
}

}  // namespace l2pd
