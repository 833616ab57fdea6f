// Memory-bound kernels of the denoising step: embedding + RMSNorm, RMSNorm, rotary
// embedding with the scatter of K/V into the per-sequence key/value store, the gather of
// the current block's rows with the final RMSNorm, and the state set-up of Algorithm 2.
#include "common.cuh"

namespace l2pd {

namespace {

__device__ __forceinline__ float block_sum(float v, float *red) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float t = (l < nw) ? red[l] : 0.f;
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  return t;
}

// x[row,:] = emb[token,:];  n[row,:] = x * g / sqrt(mean(x^2) + eps)
template <typename T>
__global__ void embed_rmsnorm_kernel(const int32_t *tokens, int64_t tok_stride, const SeqMeta *meta,
                                     const int32_t *row_slot, const T *emb, const float *gain,
                                     float eps, float *x, T *n, int d) {
  __shared__ float red[32];
  int row = blockIdx.x;
  SeqMeta m = meta[row_slot[row]];
  int pos = m.pos0 + (row - m.row0);
  int tok = tokens[(int64_t)m.seq * tok_stride + pos];
  const T *e = emb + (int64_t)tok * d;
  float *xr = x + (int64_t)row * d;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v = to_f32(e[i]);
    xr[i] = v;
    ss += v * v;
  }
  float tot = block_sum(ss, red);
  float inv = 1.0f / sqrtf(tot / (float)d + eps);
  T *nr = n + (int64_t)row * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    nr[i] = from_f32<T>(to_f32(e[i]) * gain[i] * inv);
}

template <typename T>
__global__ void rmsnorm_kernel(const float *x, const float *gain, float eps, T *n, int d) {
  __shared__ float red[32];
  int row = blockIdx.x;
  const float4 *xr = reinterpret_cast<const float4 *>(x + (int64_t)row * d);
  int d4 = d >> 2;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d4; i += blockDim.x) {
    float4 v = xr[i];
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  float tot = block_sum(ss, red);
  float inv = 1.0f / sqrtf(tot / (float)d + eps);
  const float4 *g4 = reinterpret_cast<const float4 *>(gain);
  T *nr = n + (int64_t)row * d;
  for (int i = threadIdx.x; i < d4; i += blockDim.x) {
    float4 v = xr[i];
    float4 g = g4[i];
    nr[4 * i + 0] = from_f32<T>(v.x * g.x * inv);
    nr[4 * i + 1] = from_f32<T>(v.y * g.y * inv);
    nr[4 * i + 2] = from_f32<T>(v.z * g.z * inv);
    nr[4 * i + 3] = from_f32<T>(v.w * g.w * inv);
  }
}

// Rotates q and k (pair (i, i+dh/2) by the tabulated angle of the row's position) and writes
// q to the packed query buffer and k, v to the key/value store at [sequence, position].
template <typename T>
__global__ void rope_scatter_kernel(const T *qkv, const SeqMeta *meta, const int32_t *row_slot,
                                    const float2 *cs_table, T *q, T *kc, T *vc,
                                    int64_t kv_seq_stride, int H, int dh) {
  int row = blockIdx.x;
  SeqMeta m = meta[row_slot[row]];
  int pos = m.pos0 + (row - m.row0);
  int half = dh >> 1;
  int hd = H * dh;
  const T *src = qkv + (int64_t)row * 3 * hd;
  T *qd = q + (int64_t)row * hd;
  T *kd = kc + (int64_t)m.seq * kv_seq_stride + (int64_t)pos * hd;
  T *vd = vc + (int64_t)m.seq * kv_seq_stride + (int64_t)pos * hd;
  const float2 *cs = cs_table + (int64_t)pos * half;
  for (int idx = threadIdx.x; idx < H * half; idx += blockDim.x) {
    int h = idx / half, i = idx - h * half;
    float2 c = cs[i];
    int a = h * dh + i, b = a + half;
    float q1 = to_f32(src[a]), q2 = to_f32(src[b]);
    qd[a] = from_f32<T>(q1 * c.x - q2 * c.y);
    qd[b] = from_f32<T>(q2 * c.x + q1 * c.y);
    float k1 = to_f32(src[hd + a]), k2 = to_f32(src[hd + b]);
    kd[a] = from_f32<T>(k1 * c.x - k2 * c.y);
    kd[b] = from_f32<T>(k2 * c.x + k1 * c.y);
    vd[a] = src[2 * hd + a];
    vd[b] = src[2 * hd + b];
  }
}

// Row r = slot*s + j of nf gets RMSNorm(x[row of block position j of that sequence]); rows whose
// position lies beyond L_eff, and the padding rows up to rows_padded, are zero.
template <typename T>
__global__ void final_norm_gather_kernel(const float *x, const SeqMeta *meta, const float *gain,
                                         float eps, T *nf, int n_slots, int s, int d) {
  __shared__ float red[32];
  int r = blockIdx.x;
  int slot = r / s, j = r - slot * s;
  T *out = nf + (int64_t)r * d;
  bool live = false;
  SeqMeta m;
  if (slot < n_slots) {
    m = meta[slot];
    live = j < m.n_blk_rows;
  }
  if (!live) {
    for (int i = threadIdx.x; i < d; i += blockDim.x) out[i] = from_f32<T>(0.f);
    return;
  }
  int row = m.row0 + (m.blk_start - m.pos0) + j;
  const float *xr = x + (int64_t)row * d;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) { float v = xr[i]; ss += v * v; }
  float tot = block_sum(ss, red);
  float inv = 1.0f / sqrtf(tot / (float)d + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x) out[i] = from_f32<T>(xr[i] * gain[i] * inv);
}

__global__ void build_row_map_kernel(const SeqMeta *meta, int32_t *row_slot) {
  SeqMeta m = meta[blockIdx.x];
  for (int i = threadIdx.x; i < m.n_rows; i += blockDim.x) row_slot[m.row0 + i] = blockIdx.x;
}

// Algorithm 2: X <- concat(prompt, [MASK]^G); all generation positions masked.
__global__ void state_reset_kernel(const int32_t *prompts, int P, int G, int vocab, int mask_id,
                                   int32_t *tokens, uint8_t *masked, SeqState s, int32_t *bad) {
  int b = blockIdx.x;
  int L = P + G;
  for (int i = threadIdx.x; i < L; i += blockDim.x) {
    int t = mask_id;
    if (i < P) {
      t = prompts[(int64_t)b * P + i];
      if (t < 0 || t >= vocab || t == mask_id) { atomicExch(bad, 1); t = 0; }
    }
    tokens[(int64_t)b * L + i] = t;
  }
  for (int i = threadIdx.x; i < G; i += blockDim.x) masked[(int64_t)b * G + i] = 1;
  if (threadIdx.x == 0) {
    s.cur_block[b] = 0; s.l_eff[b] = L; s.done[b] = 0; s.steps[b] = 0; s.eot_pos[b] = -1; s.forced[b] = 0;
  }
}

__global__ void gather_response_kernel(const int32_t *tokens, int P, int G, int32_t *out) {
  int b = blockIdx.x;
  for (int i = threadIdx.x; i < G; i += blockDim.x)
    out[(int64_t)b * G + i] = tokens[(int64_t)b * (P + G) + P + i];
}

}  // namespace

template <typename T>
cudaError_t launch_embed_rmsnorm(cudaStream_t st, const int32_t *tokens, int64_t tok_stride,
                                 const SeqMeta *meta, const int32_t *row_slot, const T *emb,
                                 const float *gain, float eps, float *x, T *n, int rows, int d) {
  embed_rmsnorm_kernel<T><<<rows, 256, 0, st>>>(tokens, tok_stride, meta, row_slot, emb, gain, eps, x, n, d);
  return cudaGetLastError();
}
template <typename T>
cudaError_t launch_rmsnorm(cudaStream_t st, const float *x, const float *gain, float eps, T *n,
                           int rows, int d) {
  rmsnorm_kernel<T><<<rows, 256, 0, st>>>(x, gain, eps, n, d);
  return cudaGetLastError();
}
template <typename T>
cudaError_t launch_rope_scatter(cudaStream_t st, const T *qkv, const SeqMeta *meta,
                                const int32_t *row_slot, const float2 *cs_table, T *q, T *kc, T *vc,
                                int64_t kv_seq_stride, int rows, int H, int dh) {
  rope_scatter_kernel<T><<<rows, 256, 0, st>>>(qkv, meta, row_slot, cs_table, q, kc, vc, kv_seq_stride, H, dh);
  return cudaGetLastError();
}
template <typename T>
cudaError_t launch_final_norm_gather(cudaStream_t st, const float *x, const SeqMeta *meta,
                                     const float *gain, float eps, T *nf, int n_slots, int s,
                                     int rows_padded, int d) {
  final_norm_gather_kernel<T><<<rows_padded, 256, 0, st>>>(x, meta, gain, eps, nf, n_slots, s, d);
  return cudaGetLastError();
}
cudaError_t launch_build_row_map(cudaStream_t st, const SeqMeta *meta, int n_slots, int32_t *row_slot) {
  build_row_map_kernel<<<n_slots, 256, 0, st>>>(meta, row_slot);
  return cudaGetLastError();
}
cudaError_t launch_state_reset(cudaStream_t st, const int32_t *prompts, int B, int P, int G, int vocab,
                               int mask_id, int32_t *tokens, uint8_t *masked, SeqState s, int32_t *bad) {
  state_reset_kernel<<<B, 256, 0, st>>>(prompts, P, G, vocab, mask_id, tokens, masked, s, bad);
  return cudaGetLastError();
}
cudaError_t launch_gather_response(cudaStream_t st, const int32_t *tokens, int B, int P, int G,
                                   int32_t *out) {
  gather_response_kernel<<<B, 256, 0, st>>>(tokens, P, G, out);
  return cudaGetLastError();
}

#define INSTANTIATE(T)                                                                              \
  template cudaError_t launch_embed_rmsnorm<T>(cudaStream_t, const int32_t *, int64_t,               \
                                               const SeqMeta *, const int32_t *, const T *,          \
                                               const float *, float, float *, T *, int, int);        \
  template cudaError_t launch_rmsnorm<T>(cudaStream_t, const float *, const float *, float, T *,     \
                                         int, int);                                                  \
  template cudaError_t launch_rope_scatter<T>(cudaStream_t, const T *, const SeqMeta *,              \
                                              const int32_t *, const float2 *, T *, T *, T *,        \
                                              int64_t, int, int, int);                               \
  template cudaError_t launch_final_norm_gather<T>(cudaStream_t, const float *, const SeqMeta *,     \
                                                   const float *, float, T *, int, int, int, int);
INSTANTIATE(float)
INSTANTIATE(bf16)

}  // namespace l2pd
