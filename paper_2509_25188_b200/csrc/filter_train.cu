// Filter training, stage 2 of Algorithm 1: minimise Eq. 6, the mean binary cross-entropy between
// sigmoid(f_theta(conf)) and the EGP targets, over theta = (W1, b1, W2, b2) of the two-layer filter
// (Section 3.2; 2 * (s*s + s) parameters) with AdamW (Section 4.1: learning rate 0.001).
//
// One update = two launches:
//   filter_grad_kernel   every block walks tiles of 32 samples: forward (pre, h, z), dz = sigmoid(z) - y,
//                        dh = dz W2, dpre = dh [pre > 0], and adds dz^T h, dpre^T c and the bias sums into
//                        accumulators its threads own; a block ends by writing its sums (not yet divided by
//                        the batch's element count) and its loss sum to its own row of `gpart`;
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
  const float *theta;      // packed: W1 [s*s], b1 [s], W2 [s*s], b2 [s]
  float *gpart;            // [gridDim.x, P + 1]: gradient sums, then the loss sum
};

__global__ void __launch_bounds__(GRAD_THREADS) filter_grad_kernel(GradArgs a) {
  extern __shared__ float sm[];
  const int s = a.s, sp = s + 1;     // padded row stride: rows read side by side fall into different banks
  float *W1 = sm;                    // [s][sp]
  float *W2 = W1 + s * sp;           // [s][sp]
  float *b1 = W2 + s * sp;           // [s]
  float *b2 = b1 + s;                // [s]
  float *Ct = b2 + s;                // [TB][sp] inputs of the tile
  float *Ht = Ct + TB * sp;          // [TB][sp] hidden activations
  float *Zt = Ht + TB * sp;          // [TB][sp] dz
  float *Pt = Zt + TB * sp;          // [TB][sp] pre-activations, then dpre
  __shared__ float red[GRAD_THREADS / 32];

  grid_dep_launch();
  grid_dep_wait();
  const int tid = threadIdx.x;
  const int P = 2 * (s * s + s);
  for (int e = tid; e < s * s; e += GRAD_THREADS) {
    W1[(e / s) * sp + e % s] = a.theta[e];
    W2[(e / s) * sp + e % s] = a.theta[s * s + s + e];
  }
  if (tid < s) { b1[tid] = a.theta[s * s + tid]; b2[tid] = a.theta[2 * s * s + s + tid]; }

  float acc1[MAX_OWN], acc2[MAX_OWN];
#pragma unroll
  for (int k = 0; k < MAX_OWN; ++k) { acc1[k] = 0.f; acc2[k] = 0.f; }
  float gb1 = 0.f, gb2 = 0.f, loss = 0.f;

  const int64_t n_tiles = (a.n + TB - 1) / TB;
  for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const int64_t base = a.n0 + tile * TB;
    const int rows = (int)((a.n - tile * TB) < TB ? (a.n - tile * TB) : TB);
    __syncthreads();                                   // the previous tile's buffers are no longer read
    for (int e = tid; e < TB * s; e += GRAD_THREADS) {
      const int n = e / s, i = e - n * s;
      Ct[n * sp + i] = n < rows ? a.C[(base + n) * s + i] : 0.f;
    }
    __syncthreads();
    for (int o = tid; o < TB * s; o += GRAD_THREADS) {   // pre = W1 c + b1, h = relu(pre)
      const int n = o / s, j = o - n * s;
      float v = b1[j];
      for (int i = 0; i < s; ++i) v = fmaf(W1[j * sp + i], Ct[n * sp + i], v);
      Pt[n * sp + j] = v;
      Ht[n * sp + j] = fmaxf(v, 0.f);
    }
    __syncthreads();
    for (int o = tid; o < TB * s; o += GRAD_THREADS) {   // z = W2 h + b2; dz and the loss of Eq. 6
      const int n = o / s, j = o - n * s;
      float z = b2[j];
      for (int i = 0; i < s; ++i) z = fmaf(W2[j * sp + i], Ht[n * sp + i], z);
      float dz = 0.f;
      if (n < rows) {
        const float y = (float)a.Y[(base + n) * s + j];
        dz = 1.0f / (1.0f + expf(-z)) - y;
        loss += fmaxf(z, 0.f) - z * y + log1pf(expf(-fabsf(z)));
      }
      Zt[n * sp + j] = dz;
    }
    __syncthreads();
    for (int o = tid; o < TB * s; o += GRAD_THREADS) {   // dpre = (dz W2) [pre > 0]
      const int n = o / s, i = o - n * s;
      float v = 0.f;
      for (int j = 0; j < s; ++j) v = fmaf(Zt[n * sp + j], W2[j * sp + i], v);
      Pt[n * sp + i] = Pt[n * sp + i] > 0.f ? v : 0.f;   // each thread replaces the pre-activation it alone reads
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < MAX_OWN; ++k) {                  // dW2 += dz^T h, dW1 += dpre^T c
      const int e = tid + k * GRAD_THREADS;
      if (e < s * s) {
        const int j = e / s, i = e - j * s;
        float v1 = acc1[k], v2 = acc2[k];
        for (int n = 0; n < TB; ++n) {
          v2 = fmaf(Zt[n * sp + j], Ht[n * sp + i], v2);
          v1 = fmaf(Pt[n * sp + j], Ct[n * sp + i], v1);
        }
        acc1[k] = v1; acc2[k] = v2;
      }
    }
    if (tid < s) {
      for (int n = 0; n < TB; ++n) { gb2 += Zt[n * sp + tid]; gb1 += Pt[n * sp + tid]; }
    }
  }

  float *out = a.gpart + (int64_t)blockIdx.x * (P + 1);
#pragma unroll
  for (int k = 0; k < MAX_OWN; ++k) {
    const int e = tid + k * GRAD_THREADS;
    if (e < s * s) { out[e] = acc1[k]; out[s * s + s + e] = acc2[k]; }
  }
  if (tid < s) { out[s * s + tid] = gb1; out[2 * s * s + s + tid] = gb2; }
  for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
  if ((tid & 31) == 0) red[tid >> 5] = loss;
  __syncthreads();
  if (tid == 0) {
    float t = 0.f;
    for (int w = 0; w < GRAD_THREADS / 32; ++w) t += red[w];
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
    // the rows are added in block order whatever the batching of the loads: eight loads in flight, then eight adds
    float g = 0.f;
    int b = 0;
    for (; b + 8 <= a.n_blocks; b += 8) {
      float t[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) t[i] = a.gpart[(int64_t)(b + i) * (a.P + 1) + p];
#pragma unroll
      for (int i = 0; i < 8; ++i) g += t[i];
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

size_t filter_grad_smem(int s) { return sizeof(float) * (size_t)(2 * s * (s + 1) + 2 * s + 4 * TB * (s + 1)); }

cudaError_t launch_filter_update(cudaStream_t st, const float *C, const uint8_t *Y, int64_t n0, int64_t n, int s,
                                 float *theta, float *m, float *v, float *gpart, int grid, const FilterTrainHyper &h,
                                 double bc1, double bc2, float *loss_out) {
  static bool attr = false;
  if (!attr) {
    cudaError_t e = cudaFuncSetAttribute(filter_grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)filter_grad_smem(MAX_S));
    if (e != cudaSuccess) return e;
    attr = true;
  }
  const int64_t n_tiles = (n + TB - 1) / TB;
  const int blocks = (int)(n_tiles < grid ? n_tiles : grid);
  GradArgs g{C, Y, n0, n, s, theta, gpart};
  cudaError_t e = launch_kernel(filter_grad_kernel, dim3(blocks), dim3(GRAD_THREADS), filter_grad_smem(s), st, g);
  if (e != cudaSuccess) return e;
  AdamArgs a{};
  a.gpart = gpart; a.n_blocks = blocks; a.P = 2 * (s * s + s);
  a.inv_count = (float)(1.0 / ((double)n * s));
  a.lr = h.lr; a.beta1 = h.beta1; a.beta2 = h.beta2; a.eps = h.eps; a.weight_decay = h.weight_decay;
  a.bc1 = (float)bc1; a.bc2 = (float)bc2;
  a.theta = theta; a.m = m; a.v = v; a.loss_out = loss_out;
  return launch_kernel(filter_adamw_kernel, dim3((a.P + 1 + ADAM_THREADS - 1) / ADAM_THREADS), dim3(ADAM_THREADS), 0, st, a);
}

}  // namespace l2pd
