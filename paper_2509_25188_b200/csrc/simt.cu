// CUDA-core kernels: the GEMM and attention of fp32 configurations (tcgen05 has no fp32
// kind, and TF32 would not reach 1e-4 relative accuracy), written for correctness on small
// models.  The same templates instantiate for bf16 storage as an independent cross-check
// of the tensor-core kernels.
#include "common.cuh"

namespace l2pd {

namespace {

constexpr int BM = 64, BN = 64, BK = 16;

// C[M,N] = A[M,K] * W[N,K]^T with fp32 accumulation in k order; 256 threads, 4x4 outputs each.
//   EPI_STORE      C (T)    = acc
//   EPI_RESIDUAL   X (fp32) += acc
//   EPI_SWIGLU     H (T)    = silu(acc_gate) * acc_up  (W = gate rows, W2 = up rows)
//   EPI_STORE_F32  C (fp32) = acc + bias[col]
template <typename T, int EPI>
__global__ void __launch_bounds__(256) simt_gemm_kernel(const T *__restrict__ A, const T *__restrict__ W,
                                                        const T *__restrict__ W2, void *Cv,
                                                        const float *__restrict__ bias, int M, int N, int K) {
  grid_dep_launch();
  grid_dep_wait();
  __shared__ float As[BK][BM + 1];
  __shared__ float Ws[BK][BN + 1];
  __shared__ float W2s[EPI == EPI_SWIGLU ? BK : 1][BN + 1];
  int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  float acc[4][4] = {}, acc2[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += BK) {
    for (int i = threadIdx.x; i < BM * BK; i += 256) {
      int r = i / BK, c = i - r * BK;
      int gm = m0 + r, gk = k0 + c;
      As[c][r] = (gm < M && gk < K) ? to_f32(A[(int64_t)gm * K + gk]) : 0.f;
      int gn = n0 + r;
      Ws[c][r] = (gn < N && gk < K) ? to_f32(W[(int64_t)gn * K + gk]) : 0.f;
      if (EPI == EPI_SWIGLU) W2s[c][r] = (gn < N && gk < K) ? to_f32(W2[(int64_t)gn * K + gk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[4], b[4], b2[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        a[i] = As[k][ty * 4 + i];
        b[i] = Ws[k][tx * 4 + i];
        if (EPI == EPI_SWIGLU) b2[i] = W2s[k][tx * 4 + i];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
          if (EPI == EPI_SWIGLU) acc2[i][j] = fmaf(a[i], b2[j], acc2[i][j]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      int64_t o = (int64_t)gm * N + gn;
      float v = acc[i][j];
      if (EPI == EPI_STORE) {
        reinterpret_cast<T *>(Cv)[o] = from_f32<T>(v);
      } else if (EPI == EPI_RESIDUAL) {
        reinterpret_cast<float *>(Cv)[o] += v;
      } else if (EPI == EPI_SWIGLU) {
        float sg = v / (1.0f + expf(-v));
        reinterpret_cast<T *>(Cv)[o] = from_f32<T>(sg * acc2[i][j]);
      } else {
        reinterpret_cast<float *>(Cv)[o] = v + (bias ? bias[gn] : 0.f);
      }
    }
  }
}

// One block per (query row, head): scores over all visible keys, softmax, weighted sum of values.
// No causal mask: every query sees keys [0, kv_len) of its own sequence.
template <typename T>
__global__ void simt_attention_kernel(const T *__restrict__ q, const T *__restrict__ kc,
                                      const T *__restrict__ vc, const SeqMeta *meta,
                                      const int32_t *row_slot, T *out, int64_t kv_seq_stride, int H,
                                      int dh) {
  grid_dep_launch();
  grid_dep_wait();
  extern __shared__ float sm[];
  float *qs = sm;          // [dh]
  float *sc = sm + dh;     // [kv_len]
  __shared__ float red[32];
  int row = blockIdx.x, h = blockIdx.y;
  SeqMeta m = meta[row_slot[row]];
  int hd = H * dh;
  const T *qr = q + (int64_t)row * hd + h * dh;
  for (int i = threadIdx.x; i < dh; i += blockDim.x) qs[i] = to_f32(qr[i]);
  __syncthreads();
  const T *kb = kc + (int64_t)m.seq * kv_seq_stride + h * dh;
  const T *vb = vc + (int64_t)m.seq * kv_seq_stride + h * dh;
  float scale = 1.0f / sqrtf((float)dh);
  float mx = -INFINITY;
  for (int j = threadIdx.x; j < m.kv_len; j += blockDim.x) {
    const T *kr = kb + (int64_t)j * hd;
    float a = 0.f;
    for (int c = 0; c < dh; ++c) a = fmaf(qs[c], to_f32(kr[c]), a);
    a *= scale;
    sc[j] = a;
    mx = fmaxf(mx, a);
  }
  int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (l == 0) red[w] = mx;
  __syncthreads();
  mx = (l < nw) ? red[l] : -INFINITY;
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float sum = 0.f;
  for (int j = threadIdx.x; j < m.kv_len; j += blockDim.x) {
    float e = expf(sc[j] - mx);
    sc[j] = e;
    sum += e;
  }
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  __syncthreads();
  if (l == 0) red[w] = sum;
  __syncthreads();
  sum = (l < nw) ? red[l] : 0.f;
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  float inv = 1.0f / sum;
  T *orow = out + (int64_t)row * hd + h * dh;
  for (int c = threadIdx.x; c < dh; c += blockDim.x) {
    float a = 0.f;
    for (int j = 0; j < m.kv_len; ++j) a = fmaf(sc[j], to_f32(vb[(int64_t)j * hd + c]), a);
    orow[c] = from_f32<T>(a * inv);
  }
}

// Per-row max, sum of exp and argmax (lowest id on ties) of stored fp32 logits: one tile.
__global__ void row_softmax_partials_kernel(const float *logits, int V, float *part_m, float *part_s,
                                            int32_t *part_i) {
  grid_dep_launch();
  grid_dep_wait();
  __shared__ float rm[32];
  __shared__ int ri[32];
  __shared__ float rs[32];
  int r = blockIdx.x;
  const float *row = logits + (int64_t)r * V;
  float mx = -INFINITY;
  int ix = 0x7fffffff;
  for (int v = threadIdx.x; v < V; v += blockDim.x) {
    float a = row[v];
    if (a > mx) { mx = a; ix = v; }
  }
  int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
  for (int o = 16; o > 0; o >>= 1) {
    float om = __shfl_xor_sync(0xffffffffu, mx, o);
    int oi = __shfl_xor_sync(0xffffffffu, ix, o);
    if (om > mx || (om == mx && oi < ix)) { mx = om; ix = oi; }
  }
  if (l == 0) { rm[w] = mx; ri[w] = ix; }
  __syncthreads();
  mx = (l < nw) ? rm[l] : -INFINITY;
  ix = (l < nw) ? ri[l] : 0x7fffffff;
  for (int o = 16; o > 0; o >>= 1) {
    float om = __shfl_xor_sync(0xffffffffu, mx, o);
    int oi = __shfl_xor_sync(0xffffffffu, ix, o);
    if (om > mx || (om == mx && oi < ix)) { mx = om; ix = oi; }
  }
  float sum = 0.f;
  for (int v = threadIdx.x; v < V; v += blockDim.x) sum += expf(row[v] - mx);
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (l == 0) rs[w] = sum;
  __syncthreads();
  sum = (l < nw) ? rs[l] : 0.f;
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (threadIdx.x == 0) { part_m[r] = mx; part_s[r] = sum; part_i[r] = ix; }
}

}  // namespace

template <typename T>
cudaError_t launch_simt_gemm(cudaStream_t st, int epi, const T *A, const T *W, const T *W2, void *C,
                             const float *bias, int M, int N, int K) {
  dim3 grid(ceil_div(N, BN), ceil_div(M, BM));
  switch (epi) {
    case EPI_STORE: return launch_kernel(simt_gemm_kernel<T, EPI_STORE>, grid, dim3(256), 0, st, A, W, W2, C, bias, M, N, K);
    case EPI_RESIDUAL: return launch_kernel(simt_gemm_kernel<T, EPI_RESIDUAL>, grid, dim3(256), 0, st, A, W, W2, C, bias, M, N, K);
    case EPI_SWIGLU: return launch_kernel(simt_gemm_kernel<T, EPI_SWIGLU>, grid, dim3(256), 0, st, A, W, W2, C, bias, M, N, K);
    case EPI_STORE_F32: return launch_kernel(simt_gemm_kernel<T, EPI_STORE_F32>, grid, dim3(256), 0, st, A, W, W2, C, bias, M, N, K);
    default: return cudaErrorInvalidValue;
  }
}

template <typename T>
cudaError_t launch_simt_attention(cudaStream_t st, const T *q, const T *kc, const T *vc,
                                  const SeqMeta *meta, const int32_t *row_slot, T *out,
                                  int64_t kv_seq_stride, int rows, int H, int dh, int max_kv) {
  size_t smem = (size_t)(dh + max_kv) * sizeof(float);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(simt_attention_kernel<T>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  return launch_kernel(simt_attention_kernel<T>, dim3(rows, H), dim3(128), smem, st, q, kc, vc, meta, row_slot, out,
                       kv_seq_stride, H, dh);
}

cudaError_t launch_row_softmax_partials(cudaStream_t st, const float *logits, int R, int V,
                                        float *part_m, float *part_s, int32_t *part_i) {
  return launch_kernel(row_softmax_partials_kernel, dim3(R), dim3(256), 0, st, logits, V, part_m, part_s, part_i);
}

template cudaError_t launch_simt_gemm<float>(cudaStream_t, int, const float *, const float *,
                                             const float *, void *, const float *, int, int, int);
template cudaError_t launch_simt_gemm<bf16>(cudaStream_t, int, const bf16 *, const bf16 *, const bf16 *,
                                            void *, const float *, int, int, int);
template cudaError_t launch_simt_attention<float>(cudaStream_t, const float *, const float *,
                                                  const float *, const SeqMeta *, const int32_t *,
                                                  float *, int64_t, int, int, int, int);
template cudaError_t launch_simt_attention<bf16>(cudaStream_t, const bf16 *, const bf16 *, const bf16 *,
                                                 const SeqMeta *, const int32_t *, bf16 *, int64_t, int,
                                                 int, int, int);

}  // namespace l2pd
