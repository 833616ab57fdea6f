// Filter training, stage 2 of Algorithm 1: minimise Eq. 6, the mean binary cross-entropy between
// sigmoid(f_theta(conf)) and the EGP targets, over theta = (W1, b1, W2, b2) of the two-layer filter
// (Section 3.2; 2 * (s*s + s) parameters) with AdamW (Section 4.1: learning rate 0.001).
//
// One update = two launches:
//   filter_grad_warp_kernel (s <= 32)  a warp per sample, lane j = block position j: the lane keeps row j of W1 and
//                        W2 and the accumulators of row j of both gradients in registers; the sample's vectors
//                        (c, h, dz) pass between lanes through 128-byte shared-memory slots read as broadcasts;
//   filter_grad_kernel (s > 32, or the depth variants of Section 4.4: 1 to 4 layers)  every block walks tiles of
//                        32 samples: forward through the layers, dz = sigmoid(z) - y, then layer by layer
//                        downwards dW_k += delta_k^T x_k, db_k += sum delta_k, delta_{k-1} = (delta_k W_k) [x_k > 0],
//                        into accumulators its threads own; a block ends by writing its sums (not yet divided
//                        by the batch's element count) and its loss sum to its own row of `gpart`;
//   filter_adamw_kernel  one thread per parameter adds the rows in block order (so a run is bit-reproducible), scales by
//                        1 / (samples * s) and applies AdamW: decoupled weight decay, bias-corrected moments.
// The whole problem (a few thousand parameters, samples of s floats) lives in shared memory and L2; the
// arithmetic is fp32 on CUDA cores: K = s <= 64 is far too short a contraction for the tensor cores to matter.
#include "common.cuh"

namespace l2pd {

namespace {

constexpr int TB = 32;               // samples per tile
constexpr int GRAD_THREADS = 512;
constexpr int MAX_S = 64;
constexpr int MAX_OWN = (MAX_S * MAX_S + GRAD_THREADS - 1) / GRAD_THREADS;   // accumulator elements per thread and matrix

struct GradArgs {
  const float *C;          // [N, s] filter inputs
  const uint8_t *Y;        // [N, s] targets (0 / 1)
  int64_t n0, n;           // the batch: samples [n0, n0 + n)
  int s;
  int n_layers;            // 1 .. 4 Linear(s, s) layers, ReLU between consecutive layers
  const float *theta;      // packed per layer: W_k [s*s], b_k [s]
  float *gpart;            // [gridDim.x, P + 1]: gradient sums, then the loss sum
};

constexpr int MAX_LAYERS = 4;

// Any depth, any s <= 64: every block walks tiles of 32 samples held in shared memory.
__global__ void __launch_bounds__(GRAD_THREADS) filter_grad_kernel(GradArgs a) {
  extern __shared__ float sm[];
  const int s = a.s, sp = s + 1, L = a.n_layers;   // padded row stride: rows read side by side fall into different banks
  float *W = sm;                      // [L][s][sp]
  float *Bv = W + L * s * sp;         // [L][s]
  float *X = Bv + L * s;              // [L][TB][sp]: X[0] the inputs, X[k] = relu(output of layer k - 1)
  float *D0 = X + L * TB * sp;        // [TB][sp] delta of the layer being differentiated
  float *D1 = D0 + TB * sp;           // [TB][sp] delta of the layer below
  __shared__ float red[GRAD_THREADS / 32];

  grid_dep_launch();
  grid_dep_wait();
  const int tid = threadIdx.x;
  const int per = s * s + s, P = L * per;
  for (int k = 0; k < L; ++k) {
    for (int e = tid; e < s * s; e += GRAD_THREADS) W[(k * s + e / s) * sp + e % s] = a.theta[k * per + e];
    if (tid < s) Bv[k * s + tid] = a.theta[k * per + s * s + tid];
  }

  float acc[MAX_LAYERS][MAX_OWN], gb[MAX_LAYERS];
#pragma unroll
  for (int k = 0; k < MAX_LAYERS; ++k) {
    gb[k] = 0.f;
#pragma unroll
    for (int q = 0; q < MAX_OWN; ++q) acc[k][q] = 0.f;
  }
  float loss = 0.f;

  const int64_t n_tiles = (a.n + TB - 1) / TB;
  for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const int64_t base = a.n0 + tile * TB;
    const int rows = (int)((a.n - tile * TB) < TB ? (a.n - tile * TB) : TB);
    __syncthreads();                                   // the previous tile's buffers are no longer read
    for (int e = tid; e < TB * s; e += GRAD_THREADS) {
      const int n = e / s, i = e - n * s;
      X[n * sp + i] = n < rows ? a.C[(base + n) * s + i] : 0.f;
    }
    __syncthreads();
    // forward: layer k maps X[k] to X[k + 1] = relu(.), the last layer to dz = sigmoid(z) - y in D0
    for (int k = 0; k < L; ++k) {
      const float *xin = X + k * TB * sp, *wk = W + k * s * sp;
      for (int o = tid; o < TB * s; o += GRAD_THREADS) {
        const int n = o / s, j = o - n * s;
        float v = Bv[k * s + j];
        for (int i = 0; i < s; ++i) v = fmaf(wk[j * sp + i], xin[n * sp + i], v);
        if (k + 1 < L) {
          X[(k + 1) * TB * sp + n * sp + j] = fmaxf(v, 0.f);
        } else {
          float dz = 0.f;
          if (n < rows) {
            const float y = (float)a.Y[(base + n) * s + j];
            dz = 1.0f / (1.0f + expf(-v)) - y;
            loss += fmaxf(v, 0.f) - v * y + log1pf(expf(-fabsf(v)));
          }
          D0[n * sp + j] = dz;
        }
      }
      __syncthreads();
    }
    // backward: dW_k += delta_k^T X[k], db_k += sum delta_k, delta_{k-1} = (delta_k W_k) [X[k] > 0]
    float *dcur = D0, *dnxt = D1;
#pragma unroll
    for (int kk = 0; kk < MAX_LAYERS; ++kk) {
      const int k = L - 1 - kk;
      if (k < 0) break;
      const float *xin = X + k * TB * sp, *wk = W + k * s * sp;
#pragma unroll
      for (int q = 0; q < MAX_OWN; ++q) {
        const int e = tid + q * GRAD_THREADS;
        if (e < s * s) {
          const int j = e / s, i = e - j * s;
          float v = acc[kk][q];
          for (int n = 0; n < TB; ++n) v = fmaf(dcur[n * sp + j], xin[n * sp + i], v);
          acc[kk][q] = v;
        }
      }
      if (tid < s) {
        float v = gb[kk];
        for (int n = 0; n < TB; ++n) v += dcur[n * sp + tid];
        gb[kk] = v;
      }
      if (k > 0) {
        for (int o = tid; o < TB * s; o += GRAD_THREADS) {
          const int n = o / s, i = o - n * s;
          float v = 0.f;
          for (int j = 0; j < s; ++j) v = fmaf(dcur[n * sp + j], wk[j * sp + i], v);
          dnxt[n * sp + i] = xin[n * sp + i] > 0.f ? v : 0.f;
        }
      }
      __syncthreads();
      float *t = dcur; dcur = dnxt; dnxt = t;
    }
  }

  float *out = a.gpart + (int64_t)blockIdx.x * (P + 1);
#pragma unroll
  for (int kk = 0; kk < MAX_LAYERS; ++kk) {       // acc[kk] belongs to layer L - 1 - kk
    const int k = L - 1 - kk;
    if (k < 0) break;
#pragma unroll
    for (int q = 0; q < MAX_OWN; ++q) {
      const int e = tid + q * GRAD_THREADS;
      if (e < s * s) out[k * per + e] = acc[kk][q];
    }
    if (tid < s) out[k * per + s * s + tid] = gb[kk];
  }
  for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
  if ((tid & 31) == 0) red[tid >> 5] = loss;
  __syncthreads();
  if (tid == 0) {
    float t = 0.f;
    for (int w = 0; w < GRAD_THREADS / 32; ++w) t += red[w];
    out[P] = t;
  }
}

// ---- s <= 32: a warp per sample ------------------------------------------------------------------------------
constexpr int WG_WARPS = 8;
constexpr int WG_ROW = 33;   // padded row of the W2 copy that is read by columns

__global__ void __launch_bounds__(WG_WARPS * 32) filter_grad_warp_kernel(GradArgs a) {
  extern __shared__ __align__(16) float wsm[];
  float *W2s = wsm;                               // [32][33], zero beyond s
  float *vc = W2s + 32 * WG_ROW;                  // [warps][32]; 32 * 33 floats = 4224 bytes, a multiple of 16
  float *vh = vc + WG_WARPS * 32;
  float *vd = vh + WG_WARPS * 32;
  float *red = vd + WG_WARPS * 32;                // [warps][2 * 1024 + 64] at the end of the kernel

  grid_dep_launch();
  grid_dep_wait();
  const int s = a.s, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int P = 2 * (s * s + s);
  for (int e = threadIdx.x; e < 32 * 32; e += blockDim.x) {
    const int j = e >> 5, i = e & 31;
    W2s[j * WG_ROW + i] = (j < s && i < s) ? a.theta[s * s + s + j * s + i] : 0.f;
  }
  float w1[32], w2[32], acc1[32], acc2[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    const bool in = lane < s && i < s;
    w1[i] = in ? a.theta[lane * s + i] : 0.f;
    w2[i] = in ? a.theta[s * s + s + lane * s + i] : 0.f;
    acc1[i] = 0.f; acc2[i] = 0.f;
  }
  const float b1 = lane < s ? a.theta[s * s + lane] : 0.f, b2 = lane < s ? a.theta[2 * s * s + s + lane] : 0.f;
  float gb1 = 0.f, gb2 = 0.f, loss = 0.f;
  __syncthreads();

  float *mc = vc + warp * 32, *mh = vh + warp * 32, *md = vd + warp * 32;
  const int64_t stride = (int64_t)gridDim.x * WG_WARPS;
  // the next sample's row is requested before the current one is worked on (a warp has no other loads to hide it behind)
  int64_t n = (int64_t)blockIdx.x * WG_WARPS + warp;
  float c_nx = 0.f, y_nx = 0.f;
  if (n < a.n && lane < s) { c_nx = a.C[(a.n0 + n) * s + lane]; y_nx = (float)a.Y[(a.n0 + n) * s + lane]; }
  for (; n < a.n; n += stride) {
    const float c = c_nx, y = y_nx;
    if (n + stride < a.n && lane < s) {
      const int64_t row = (a.n0 + n + stride) * s;
      c_nx = a.C[row + lane]; y_nx = (float)a.Y[row + lane];
    }
    mc[lane] = c;
    __syncwarp();
    // the dot products run as four interleaved partial sums (a single chain of 32 dependent multiply-adds would
    // leave the two warps a scheduler has here waiting on latency); the order of the additions is fixed
    float p0 = b1, p1 = 0.f, p2 = 0.f, p3 = 0.f;           // pre_j = W1[j,:] c + b1_j
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float4 v = *reinterpret_cast<const float4 *>(mc + 4 * q);
      p0 = fmaf(w1[4 * q], v.x, p0); p1 = fmaf(w1[4 * q + 1], v.y, p1);
      p2 = fmaf(w1[4 * q + 2], v.z, p2); p3 = fmaf(w1[4 * q + 3], v.w, p3);
    }
    const float pre = (p0 + p1) + (p2 + p3);
    const float h = fmaxf(pre, 0.f);
    mh[lane] = lane < s ? h : 0.f;
    __syncwarp();
    p0 = b2; p1 = 0.f; p2 = 0.f; p3 = 0.f;                 // z_j = W2[j,:] h + b2_j
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float4 v = *reinterpret_cast<const float4 *>(mh + 4 * q);
      p0 = fmaf(w2[4 * q], v.x, p0); p1 = fmaf(w2[4 * q + 1], v.y, p1);
      p2 = fmaf(w2[4 * q + 2], v.z, p2); p3 = fmaf(w2[4 * q + 3], v.w, p3);
    }
    const float z = (p0 + p1) + (p2 + p3);
    float dz = 0.f;
    if (lane < s) {
      dz = 1.0f / (1.0f + expf(-z)) - y;
      loss += fmaxf(z, 0.f) - z * y + log1pf(expf(-fabsf(z)));
    }
    md[lane] = dz;
    __syncwarp();
    p0 = 0.f; p1 = 0.f; p2 = 0.f; p3 = 0.f;                // dh_i = sum_j W2[j, i] dz_j  (lane = i)
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float4 v = *reinterpret_cast<const float4 *>(md + 4 * q);
      p0 = fmaf(W2s[(4 * q) * WG_ROW + lane], v.x, p0); p1 = fmaf(W2s[(4 * q + 1) * WG_ROW + lane], v.y, p1);
      p2 = fmaf(W2s[(4 * q + 2) * WG_ROW + lane], v.z, p2); p3 = fmaf(W2s[(4 * q + 3) * WG_ROW + lane], v.w, p3);
    }
    const float dh = (p0 + p1) + (p2 + p3);
    const float dpre = pre > 0.f ? dh : 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) {                          // rows j of dW2 += dz_j h, of dW1 += dpre_j c
      const float4 vh4 = *reinterpret_cast<const float4 *>(mh + 4 * q);
      const float4 vc4 = *reinterpret_cast<const float4 *>(mc + 4 * q);
      acc2[4 * q] = fmaf(dz, vh4.x, acc2[4 * q]); acc2[4 * q + 1] = fmaf(dz, vh4.y, acc2[4 * q + 1]);
      acc2[4 * q + 2] = fmaf(dz, vh4.z, acc2[4 * q + 2]); acc2[4 * q + 3] = fmaf(dz, vh4.w, acc2[4 * q + 3]);
      acc1[4 * q] = fmaf(dpre, vc4.x, acc1[4 * q]); acc1[4 * q + 1] = fmaf(dpre, vc4.y, acc1[4 * q + 1]);
      acc1[4 * q + 2] = fmaf(dpre, vc4.z, acc1[4 * q + 2]); acc1[4 * q + 3] = fmaf(dpre, vc4.w, acc1[4 * q + 3]);
    }
    gb2 += dz; gb1 += dpre;
    __syncwarp();                                          // the slots are rewritten by the next sample
  }

  // the block's sums: every warp parks its rows, then each element is added over the warps in warp order
  float *mine = red + warp * (2 * 1024 + 64);
#pragma unroll
  for (int i = 0; i < 32; ++i) { mine[i * 32 + lane] = acc1[i]; mine[1024 + i * 32 + lane] = acc2[i]; }   // [column][row]: no bank conflicts
  mine[2048 + lane] = gb1; mine[2048 + 32 + lane] = gb2;
  for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
  __shared__ float wloss[WG_WARPS];
  if (lane == 0) wloss[warp] = loss;
  __syncthreads();
  float *out = a.gpart + (int64_t)blockIdx.x * (P + 1);
  for (int e = threadIdx.x; e < 2 * 1024 + 64; e += blockDim.x) {
    float t = 0.f;
    for (int w = 0; w < WG_WARPS; ++w) t += red[w * (2 * 1024 + 64) + e];
    if (e < 2048) {
      const int mat = e >> 10, i = (e >> 5) & 31, j = e & 31;
      if (j < s && i < s) out[mat * (s * s + s) + j * s + i] = t;
    } else {
      const int which = (e - 2048) >> 5, j = e & 31;
      if (j < s) out[which * (s * s + s) + s * s + j] = t;
    }
  }
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < WG_WARPS; ++w) t += wloss[w];
    out[P] = t;
  }
}

struct AdamArgs {
  const float *gpart;
  int n_blocks, P;
  float inv_count;                 // 1 / (samples in the batch * s)
  float lr, beta1, beta2, eps, weight_decay;
  float bc1, bc2;                  // 1 - beta1^t, 1 - beta2^t
  float *theta, *m, *v;
  float *loss_out;                 // the batch's loss, measured before this update
};

constexpr int ADAM_THREADS = 128;

__global__ void __launch_bounds__(ADAM_THREADS) filter_adamw_kernel(AdamArgs a) {
  grid_dep_launch();
  grid_dep_wait();
  const int p = blockIdx.x * ADAM_THREADS + threadIdx.x;   // one parameter per thread; entry P is the loss
  if (p <= a.P) {
    // the rows are added in block order whatever the batching of the loads: 32 loads in flight, then 32 adds
    float g = 0.f;
    int b = 0;
    for (; b + 32 <= a.n_blocks; b += 32) {
      float t[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) t[i] = a.gpart[(int64_t)(b + i) * (a.P + 1) + p];
#pragma unroll
      for (int i = 0; i < 32; ++i) g += t[i];
    }
    for (; b < a.n_blocks; ++b) g += a.gpart[(int64_t)b * (a.P + 1) + p];
    g *= a.inv_count;
    if (p == a.P) { *a.loss_out = g; return; }
    const float th = a.theta[p] * (1.0f - a.lr * a.weight_decay);
    const float m = a.beta1 * a.m[p] + (1.0f - a.beta1) * g;
    const float v = a.beta2 * a.v[p] + (1.0f - a.beta2) * g * g;
    a.m[p] = m; a.v[p] = v;
    a.theta[p] = th - a.lr * (m / a.bc1) / (sqrtf(v / a.bc2) + a.eps);
  }
}

}  // namespace

size_t filter_grad_smem(int s, int L) { return sizeof(float) * (size_t)(L * s * (s + 1) + L * s + (L + 2) * TB * (s + 1)); }
constexpr size_t WG_SMEM = sizeof(float) * (32 * WG_ROW + 3 * WG_WARPS * 32 + WG_WARPS * (2 * 1024 + 64));

cudaError_t launch_filter_update(cudaStream_t st, const float *C, const uint8_t *Y, int64_t n0, int64_t n, int s, int n_layers,
                                 float *theta, float *m, float *v, float *gpart, int grid, const FilterTrainHyper &h,
                                 double bc1, double bc2, float *loss_out) {
  if (n_layers < 1 || n_layers > MAX_LAYERS || s < 1 || s > MAX_S) return cudaErrorInvalidValue;
  GradArgs g{C, Y, n0, n, s, n_layers, theta, gpart};
  int blocks;
  cudaError_t e;
  if (s <= 32 && n_layers == 2) {
    static bool attr_w = false;
    if (!attr_w) {
      e = cudaFuncSetAttribute(filter_grad_warp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)WG_SMEM);
      if (e != cudaSuccess) return e;
      attr_w = true;
    }
    const int64_t want = (n + WG_WARPS - 1) / WG_WARPS;
    blocks = (int)(want < grid ? want : grid);
    e = launch_kernel(filter_grad_warp_kernel, dim3(blocks), dim3(WG_WARPS * 32), WG_SMEM, st, g);
  } else {
    static bool attr = false;
    if (!attr) {
      e = cudaFuncSetAttribute(filter_grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)filter_grad_smem(MAX_S, MAX_LAYERS));
      if (e != cudaSuccess) return e;
      attr = true;
    }
    const int64_t n_tiles = (n + TB - 1) / TB;
    blocks = (int)(n_tiles < grid ? n_tiles : grid);
    e = launch_kernel(filter_grad_kernel, dim3(blocks), dim3(GRAD_THREADS), filter_grad_smem(s, n_layers), st, g);
  }
  if (e != cudaSuccess) return e;
  AdamArgs a{};
  a.gpart = gpart; a.n_blocks = blocks; a.P = n_layers * (s * s + s);
  a.inv_count = (float)(1.0 / ((double)n * s));
  a.lr = h.lr; a.beta1 = h.beta1; a.beta2 = h.beta2; a.eps = h.eps; a.weight_decay = h.weight_decay;
  a.bc1 = (float)bc1; a.bc2 = (float)bc2;
  a.theta = theta; a.m = m; a.v = v; a.loss_out = loss_out;
  return launch_kernel(filter_adamw_kernel, dim3((a.P + 1 + ADAM_THREADS - 1) / ADAM_THREADS), dim3(ADAM_THREADS), 0, st, a);
}

}  // namespace l2pd
