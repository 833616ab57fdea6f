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

template <typename T> struct Vec8;
template <> struct Vec8<bf16> {
  uint4 raw;
  __device__ __forceinline__ void load(const bf16 *p) { raw = *reinterpret_cast<const uint4 *>(p); }
  __device__ __forceinline__ void store(bf16 *p) const { *reinterpret_cast<uint4 *>(p) = raw; }
  __device__ __forceinline__ float get(int i) const {
    const __nv_bfloat16 *h = reinterpret_cast<const __nv_bfloat16 *>(&raw);
    return __bfloat162float(h[i]);
  }
  __device__ __forceinline__ void set(int i, float f) {
    __nv_bfloat16 *h = reinterpret_cast<__nv_bfloat16 *>(&raw);
    h[i] = __float2bfloat16_rn(f);
  }
};
template <> struct Vec8<float> {
  float4 a, b;
  __device__ __forceinline__ void load(const float *p) {
    a = *reinterpret_cast<const float4 *>(p);
    b = *reinterpret_cast<const float4 *>(p + 4);
  }
  __device__ __forceinline__ void store(float *p) const {
    *reinterpret_cast<float4 *>(p) = a;
    *reinterpret_cast<float4 *>(p + 4) = b;
  }
  __device__ __forceinline__ float get(int i) const { return reinterpret_cast<const float *>(&a)[i]; }
  __device__ __forceinline__ void set(int i, float f) { reinterpret_cast<float *>(&a)[i] = f; }
};

// x[row,:] = emb[token,:];  n[row,:] = x * g / sqrt(mean(x^2) + eps)
template <typename T>
__global__ void embed_rmsnorm_kernel(const int32_t *tokens, int64_t tok_stride, const SeqMeta *meta,
                                     const int32_t *row_slot, const T *emb, const float *gain,
                                     float eps, float *x, T *n, int d) {
  grid_dep_launch();
  grid_dep_wait();
  __shared__ float red[32];
  int row = blockIdx.x;
  SeqMeta m = meta[row_slot[row]];
  int pos = m.pos0 + (row - m.row0);
  int tok = tokens[(int64_t)m.seq * tok_stride + pos];
  const T *e = emb + (int64_t)tok * d;
  float *xr = x + (int64_t)row * d;
  T *nr = n + (int64_t)row * d;
  float ss = 0.f;
  if ((d & 7) == 0) {
    // 8 elements per access (16 bytes of bf16 / 32 of fp32); per thread the sum runs over its chunks in order and
    // over the 8 elements of a chunk in order
    const int d8 = d >> 3;
    for (int c = threadIdx.x; c < d8; c += blockDim.x) {
      Vec8<T> v;
      v.load(e + 8 * c);
      float f[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) { f[i] = v.get(i); ss += f[i] * f[i]; }
      *reinterpret_cast<float4 *>(xr + 8 * c) = make_float4(f[0], f[1], f[2], f[3]);
      *reinterpret_cast<float4 *>(xr + 8 * c + 4) = make_float4(f[4], f[5], f[6], f[7]);
    }
    const float tot = block_sum(ss, red);
    const float inv = 1.0f / sqrtf(tot / (float)d + eps);
    for (int c = threadIdx.x; c < d8; c += blockDim.x) {
      Vec8<T> v, o;
      v.load(e + 8 * c);
      const float4 g0 = *reinterpret_cast<const float4 *>(gain + 8 * c), g1 = *reinterpret_cast<const float4 *>(gain + 8 * c + 4);
      const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) o.set(i, v.get(i) * g[i] * inv);
      o.store(nr + 8 * c);
    }
    return;
  }
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v = to_f32(e[i]);
    xr[i] = v;
    ss += v * v;
  }
  float tot = block_sum(ss, red);
  float inv = 1.0f / sqrtf(tot / (float)d + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    nr[i] = from_f32<T>(to_f32(e[i]) * gain[i] * inv);
}

__device__ __forceinline__ void store4(float *p, float a, float b, float c, float d) {
  *reinterpret_cast<float4 *>(p) = make_float4(a, b, c, d);
}
__device__ __forceinline__ void store4(bf16 *p, float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t *>(&lo);
  u.y = *reinterpret_cast<uint32_t *>(&hi);
  *reinterpret_cast<uint2 *>(p) = u;
}

// One block per row; rows up to 4 * 4 * blockDim floats stay in registers between the two passes.
// n_part > 0: the row first takes in the partial sums of a K-split projection, slice after slice, and
// the summed row is written back to x.
// NPART is a compile-time count so that all loads of a row chunk are issued before the first addition.
template <typename T, int NPART>
__global__ void __launch_bounds__(256) rmsnorm_kernel(float *x, const float *gain, float eps, T *n, int d,
                                                      const float *part, int64_t part_stride) {
  grid_dep_launch();
  grid_dep_wait();
  __shared__ float red[32];
  const int row = blockIdx.x;
  float4 *xr = reinterpret_cast<float4 *>(x + (int64_t)row * d);
  const int d4 = d >> 2;
  constexpr int CACHE = 4;
  float4 v[CACHE];
  float ss = 0.f;
  auto fetch = [&](int i) {
    float4 w = xr[i];
    if (NPART > 0) {
      float4 q[NPART > 0 ? NPART : 1];
#pragma unroll
      for (int s = 0; s < NPART; ++s) q[s] = reinterpret_cast<const float4 *>(part + s * part_stride + (int64_t)row * d)[i];
#pragma unroll
      for (int s = 0; s < NPART; ++s) { w.x += q[s].x; w.y += q[s].y; w.z += q[s].z; w.w += q[s].w; }
      xr[i] = w;
    }
    return w;
  };
#pragma unroll
  for (int k = 0; k < CACHE; ++k) {
    const int i = threadIdx.x + k * blockDim.x;
    v[k] = (i < d4) ? fetch(i) : make_float4(0.f, 0.f, 0.f, 0.f);
    ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
  }
  for (int i = threadIdx.x + CACHE * blockDim.x; i < d4; i += blockDim.x) {
    float4 w = fetch(i);
    ss += w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
  }
  const float tot = block_sum(ss, red);
  const float inv = 1.0f / sqrtf(tot / (float)d + eps);
  const float4 *g4 = reinterpret_cast<const float4 *>(gain);
  T *nr = n + (int64_t)row * d;
#pragma unroll
  for (int k = 0; k < CACHE; ++k) {
    const int i = threadIdx.x + k * blockDim.x;
    if (i < d4) {
      const float4 g = g4[i];
      store4(nr + 4 * i, v[k].x * g.x * inv, v[k].y * g.y * inv, v[k].z * g.z * inv, v[k].w * g.w * inv);
    }
  }
  for (int i = threadIdx.x + CACHE * blockDim.x; i < d4; i += blockDim.x) {
    const float4 w = xr[i];          // already summed and written back above, by this same thread
    const float4 g = g4[i];
    store4(nr + 4 * i, w.x * g.x * inv, w.y * g.y * inv, w.z * g.z * inv, w.w * g.w * inv);
  }
}

__global__ void __launch_bounds__(256) add_partials_kernel(float *x, const float *part, int n_part, int64_t part_stride,
                                                           int64_t n4) {
  grid_dep_launch();
  grid_dep_wait();
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
    float4 w = reinterpret_cast<float4 *>(x)[i];
    for (int s = 0; s < n_part; ++s) {
      const float4 q = reinterpret_cast<const float4 *>(part + s * part_stride)[i];
      w.x += q.x; w.y += q.y; w.z += q.z; w.w += q.w;
    }
    reinterpret_cast<float4 *>(x)[i] = w;
  }
}

// Rotates q and k (pair (i, i+dh/2) by the tabulated angle of the row's position) and writes
// q to the packed query buffer and k, v to the key/value store at [sequence, position].
// One work item = 8 consecutive pair indices of one head (16-byte accesses); needs dh % 16 == 0.
template <typename T>
__global__ void __launch_bounds__(256) rope_scatter_vec_kernel(const T *qkv, const SeqMeta *meta,
                                                                const int32_t *row_slot, const float2 *cs_table,
                                                                T *q, T *kc, T *vc, int64_t kv_seq_stride, int H,
                                                                int dh) {
  grid_dep_launch();
  grid_dep_wait();
  const int row = blockIdx.x;
  const SeqMeta m = meta[row_slot[row]];
  const int pos = m.pos0 + (row - m.row0);
  const int half = dh >> 1, hd = H * dh, per_head = half >> 3;
  const T *src = qkv + (int64_t)row * 3 * hd;
  T *qd = q + (int64_t)row * hd;
  T *kd = kc + (int64_t)m.seq * kv_seq_stride + (int64_t)pos * hd;
  T *vd = vc + (int64_t)m.seq * kv_seq_stride + (int64_t)pos * hd;
  const float2 *cs = cs_table + (int64_t)pos * half;
  for (int item = threadIdx.x; item < H * per_head; item += blockDim.x) {
    const int h = item / per_head, c = item - h * per_head;
    const int a = h * dh + c * 8, b = a + half;
    float2 t[8];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      *reinterpret_cast<float4 *>(&t[2 * i]) = *reinterpret_cast<const float4 *>(&cs[c * 8 + 2 * i]);
    Vec8<T> x1, x2, y1, y2;
    x1.load(src + a); x2.load(src + b);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float u = x1.get(i), w = x2.get(i);
      y1.set(i, u * t[i].x - w * t[i].y);
      y2.set(i, w * t[i].x + u * t[i].y);
    }
    y1.store(qd + a); y2.store(qd + b);
    x1.load(src + hd + a); x2.load(src + hd + b);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float u = x1.get(i), w = x2.get(i);
      y1.set(i, u * t[i].x - w * t[i].y);
      y2.set(i, w * t[i].x + u * t[i].y);
    }
    y1.store(kd + a); y2.store(kd + b);
    x1.load(src + 2 * hd + a); x2.load(src + 2 * hd + b);
    x1.store(vd + a); x2.store(vd + b);
  }
}

// Scalar form for head sizes that are not a multiple of 16.
template <typename T>
__global__ void rope_scatter_kernel(const T *qkv, const SeqMeta *meta, const int32_t *row_slot,
                                    const float2 *cs_table, T *q, T *kc, T *vc,
                                    int64_t kv_seq_stride, int H, int dh) {
  grid_dep_launch();
  grid_dep_wait();
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
  grid_dep_launch();
  grid_dep_wait();
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
  if ((d & 3) == 0) {
    // four elements per access; the row stays in registers between the two passes when it fits
    const int d4 = d >> 2;
    const float4 *x4 = reinterpret_cast<const float4 *>(xr), *g4 = reinterpret_cast<const float4 *>(gain);
    constexpr int CACHE = 4;
    float4 v[CACHE];
#pragma unroll
    for (int k = 0; k < CACHE; ++k) {
      const int i = threadIdx.x + k * blockDim.x;
      v[k] = i < d4 ? x4[i] : make_float4(0.f, 0.f, 0.f, 0.f);
      ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
    }
    for (int i = threadIdx.x + CACHE * blockDim.x; i < d4; i += blockDim.x) {
      const float4 w = x4[i];
      ss += w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
    }
    const float tot = block_sum(ss, red);
    const float inv = 1.0f / sqrtf(tot / (float)d + eps);
#pragma unroll
    for (int k = 0; k < CACHE; ++k) {
      const int i = threadIdx.x + k * blockDim.x;
      if (i < d4) { const float4 g = g4[i]; store4(out + 4 * i, v[k].x * g.x * inv, v[k].y * g.y * inv, v[k].z * g.z * inv, v[k].w * g.w * inv); }
    }
    for (int i = threadIdx.x + CACHE * blockDim.x; i < d4; i += blockDim.x) {
      const float4 w = x4[i], g = g4[i];
      store4(out + 4 * i, w.x * g.x * inv, w.y * g.y * inv, w.z * g.z * inv, w.w * g.w * inv);
    }
    return;
  }
  for (int i = threadIdx.x; i < d; i += blockDim.x) { float v = xr[i]; ss += v * v; }
  float tot = block_sum(ss, red);
  float inv = 1.0f / sqrtf(tot / (float)d + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x) out[i] = from_f32<T>(xr[i] * gain[i] * inv);
}

__global__ void build_row_map_kernel(const SeqMeta *meta, int32_t *row_slot, int32_t *row_pos) {
  grid_dep_launch();
  grid_dep_wait();
  SeqMeta m = meta[blockIdx.x];
  for (int i = threadIdx.x; i < m.n_rows; i += blockDim.x) {
    row_slot[m.row0 + i] = blockIdx.x;
    row_pos[m.row0 + i] = m.pos0 + i;
  }
}

// dst row (h, r) of the q and k parts = src row (h, r / 2 + (r odd ? dh / 2 : 0)); v rows unchanged
__global__ void permute_qkv_rows_kernel(const bf16 *src, bf16 *dst, int H, int dh, int d) {
  const int row = blockIdx.x;                 // destination row in [0, 3 * H * dh)
  const int hd = H * dh;
  int srow = row;
  if (row < 2 * hd) {
    const int part = row / hd, in = row - part * hd, h = in / dh, r = in - h * dh;
    srow = part * hd + h * dh + (r >> 1) + ((r & 1) ? (dh >> 1) : 0);
  }
  const uint4 *s = reinterpret_cast<const uint4 *>(src + (int64_t)srow * d);
  uint4 *t = reinterpret_cast<uint4 *>(dst + (int64_t)row * d);
  for (int i = threadIdx.x; i < d / 8; i += blockDim.x) t[i] = s[i];
}

// Algorithm 2: X <- concat(prompt, [MASK]^G); all generation positions masked.
__global__ void state_reset_kernel(const int32_t *prompts, int P, int G, int vocab, int mask_id,
                                   int32_t *tokens, uint8_t *masked, SeqState s, int32_t *bad) {
  grid_dep_launch();
  grid_dep_wait();
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

// Sets *bad when an id is outside [0, vocab) or is the mask token.
__global__ void check_ids_kernel(const int32_t *ids, int64_t n, int vocab, int mask_id, int32_t *bad) {
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    int t = ids[i];
    if (t < 0 || t >= vocab || t == mask_id) atomicExch(bad, 1);
  }
}

__global__ void gather_response_kernel(const int32_t *tokens, int P, int G, int32_t *out) {
  grid_dep_launch();
  grid_dep_wait();
  int b = blockIdx.x;
  for (int i = threadIdx.x; i < G; i += blockDim.x)
    out[(int64_t)b * G + i] = tokens[(int64_t)b * (P + G) + P + i];
}

}  // namespace

template <typename T>
cudaError_t launch_embed_rmsnorm(cudaStream_t st, const int32_t *tokens, int64_t tok_stride,
                                 const SeqMeta *meta, const int32_t *row_slot, const T *emb,
                                 const float *gain, float eps, float *x, T *n, int rows, int d) {
  return launch_kernel(embed_rmsnorm_kernel<T>, dim3(rows), dim3(256), 0, st, tokens, tok_stride, meta, row_slot, emb, gain, eps, x, n, d);
}
template <typename T>
cudaError_t launch_rmsnorm(cudaStream_t st, float *x, const float *gain, float eps, T *n,
                           int rows, int d, const float *part, int n_part, int64_t part_stride) {
  switch (n_part) {
    case 0: return launch_kernel(rmsnorm_kernel<T, 0>, dim3(rows), dim3(256), 0, st, x, gain, eps, n, d, part, part_stride);
    case 2: return launch_kernel(rmsnorm_kernel<T, 2>, dim3(rows), dim3(256), 0, st, x, gain, eps, n, d, part, part_stride);
    case 3: return launch_kernel(rmsnorm_kernel<T, 3>, dim3(rows), dim3(256), 0, st, x, gain, eps, n, d, part, part_stride);
    case 4: return launch_kernel(rmsnorm_kernel<T, 4>, dim3(rows), dim3(256), 0, st, x, gain, eps, n, d, part, part_stride);
    default: return cudaErrorInvalidValue;
  }
}
cudaError_t launch_add_partials(cudaStream_t st, float *x, const float *part, int n_part, int64_t part_stride, int rows, int d) {
  const int64_t n4 = (int64_t)rows * d / 4;
  const int grid = (int)((n4 + 255) / 256 < 2048 ? (n4 + 255) / 256 : 2048);
  return launch_kernel(add_partials_kernel, dim3(grid), dim3(256), 0, st, x, part, n_part, part_stride, n4);
}
template <typename T>
cudaError_t launch_rope_scatter(cudaStream_t st, const T *qkv, const SeqMeta *meta,
                                const int32_t *row_slot, const float2 *cs_table, T *q, T *kc, T *vc,
                                int64_t kv_seq_stride, int rows, int H, int dh) {
  if (dh % 16 == 0 && (H * dh) % 8 == 0)
    return launch_kernel(rope_scatter_vec_kernel<T>, dim3(rows), dim3(256), 0, st, qkv, meta, row_slot, cs_table, q, kc, vc,
                         kv_seq_stride, H, dh);
  return launch_kernel(rope_scatter_kernel<T>, dim3(rows), dim3(256), 0, st, qkv, meta, row_slot, cs_table, q, kc, vc,
                       kv_seq_stride, H, dh);
}
template <typename T>
cudaError_t launch_final_norm_gather(cudaStream_t st, const float *x, const SeqMeta *meta,
                                     const float *gain, float eps, T *nf, int n_slots, int s,
                                     int rows_padded, int d) {
  return launch_kernel(final_norm_gather_kernel<T>, dim3(rows_padded), dim3(256), 0, st, x, meta, gain, eps, nf, n_slots, s, d);
}
cudaError_t launch_build_row_map(cudaStream_t st, const SeqMeta *meta, int n_slots, int32_t *row_slot, int32_t *row_pos) {
  return launch_kernel(build_row_map_kernel, dim3(n_slots), dim3(256), 0, st, meta, row_slot, row_pos);
}
cudaError_t launch_permute_qkv_rows(cudaStream_t st, const bf16 *src, bf16 *dst, int H, int dh, int d) {
  permute_qkv_rows_kernel<<<3 * H * dh, 256, 0, st>>>(src, dst, H, dh, d);
  return cudaGetLastError();
}
cudaError_t launch_state_reset(cudaStream_t st, const int32_t *prompts, int B, int P, int G, int vocab,
                               int mask_id, int32_t *tokens, uint8_t *masked, SeqState s, int32_t *bad) {
  return launch_kernel(state_reset_kernel, dim3(B), dim3(256), 0, st, prompts, P, G, vocab, mask_id, tokens, masked, s, bad);
}
cudaError_t launch_check_ids(cudaStream_t st, const int32_t *ids, int64_t n, int vocab, int mask_id, int32_t *bad) {
  int blocks = (int)((n + 255) / 256);
  blocks = blocks < 1 ? 1 : (blocks > 592 ? 592 : blocks);
  check_ids_kernel<<<blocks, 256, 0, st>>>(ids, n, vocab, mask_id, bad);
  return cudaGetLastError();
}
cudaError_t launch_gather_response(cudaStream_t st, const int32_t *tokens, int B, int P, int G,
                                   int32_t *out) {
  return launch_kernel(gather_response_kernel, dim3(B), dim3(256), 0, st, tokens, P, G, out);
}

#define INSTANTIATE(T)                                                                              \
  template cudaError_t launch_embed_rmsnorm<T>(cudaStream_t, const int32_t *, int64_t,               \
                                               const SeqMeta *, const int32_t *, const T *,          \
                                               const float *, float, float *, T *, int, int);        \
  template cudaError_t launch_rmsnorm<T>(cudaStream_t, float *, const float *, float, T *,           \
                                         int, int, const float *, int, int64_t);                     \
  template cudaError_t launch_rope_scatter<T>(cudaStream_t, const T *, const SeqMeta *,              \
                                              const int32_t *, const float2 *, T *, T *, T *,        \
                                              int64_t, int, int, int);                               \
  template cudaError_t launch_final_norm_gather<T>(cudaStream_t, const float *, const SeqMeta *,     \
                                                   const float *, float, T *, int, int, int, int);
INSTANTIATE(float)
INSTANTIATE(bf16)

}  // namespace l2pd
