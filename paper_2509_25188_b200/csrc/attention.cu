// Bidirectional (non-causal) multi-head attention, bf16, flash style: one pass over the keys with
// a running row max and row sum, so the [queries x keys] score matrix never leaves the SM.
// Every query of a sequence sees keys [0, kv_len) of that sequence — there is no mask to apply,
// only the ragged tail of the last key tile.
//
// CTA = 4 warps x 16 query rows; key/value tiles of 64 rows double-buffered in shared memory with
// cp.async; S = Q K^T and O += P V on warp-level mma.sync m16n8k16 with fp32 accumulation; the
// probabilities are re-used from the score registers as the A operand of the second product.
#include "common.cuh"

namespace l2pd {

namespace {

constexpr int BQ = 64;    // query rows per CTA
constexpr int BKV = 64;   // keys per tile

__device__ __forceinline__ uint32_t smem_addr(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float *c, const uint32_t *a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&t);
}

// Tile rows are DH bf16 = DH/8 chunks of 16 bytes; chunk c of row r is stored at chunk c ^ (r & 7)
// so that the 8 rows an ldmatrix reads fall in different banks.
template <int DH>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return (uint32_t)(row * (DH * 2) + ((chunk ^ (row & 7)) << 4));
}

template <int DH>
__device__ __forceinline__ void load_tile(uint32_t dst, const bf16 *src, int64_t row_stride, int rows_valid,
                                          int tid) {
  constexpr int CH = DH / 8;
  for (int i = tid; i < BKV * CH; i += 128) {
    const int r = i / CH, c = i - r * CH;
    const bool ok = r < rows_valid;
    const bf16 *s = src + (int64_t)(ok ? r : 0) * row_stride + c * 8;
    cp_async16(dst + tile_off<DH>(r, c), s, ok ? 16 : 0);
  }
}

struct AttnParams {
  const bf16 *q, *kc, *vc;
  bf16 *out;
  const SeqMeta *meta;
  SeqMeta single;
  int use_single;
  int64_t q_stride, kv_row_stride, kv_seq_stride, out_stride;
  float scale_log2;
};

template <int DH>
__global__ void __launch_bounds__(128) attention_bf16_kernel(const AttnParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  constexpr int TILE_BYTES = BKV * DH * 2;
  const uint32_t sQ = smem_addr(smem);
  const uint32_t sK = sQ + BQ * DH * 2;
  const uint32_t sV = sK + 2 * TILE_BYTES;

  grid_dep_launch();
  grid_dep_wait();
  const SeqMeta m = p.use_single ? p.single : p.meta[blockIdx.z];
  const int q0 = blockIdx.x * BQ;
  if (q0 >= m.n_rows) return;
  const int h = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int q_valid = min(BQ, m.n_rows - q0);
  const int kv_len = m.kv_len;
  const int n_tiles = (kv_len + BKV - 1) / BKV;

  const bf16 *qg = p.q + (int64_t)(m.row0 + q0) * p.q_stride + h * DH;
  const bf16 *kg = p.kc + (int64_t)m.seq * p.kv_seq_stride + h * DH;
  const bf16 *vg = p.vc + (int64_t)m.seq * p.kv_seq_stride + h * DH;

  load_tile<DH>(sQ, qg, p.q_stride, q_valid, tid);
  load_tile<DH>(sK, kg, p.kv_row_stride, min(BKV, kv_len), tid);
  load_tile<DH>(sV, vg, p.kv_row_stride, min(BKV, kv_len), tid);
  cp_commit();

  uint32_t qf[DH / 16][4];
  float o[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

  for (int j = 0; j < n_tiles; ++j) {
    const int buf = j & 1;
    if (j + 1 < n_tiles) {
      const int k0n = (j + 1) * BKV;
      load_tile<DH>(sK + (buf ^ 1) * TILE_BYTES, kg + (int64_t)k0n * p.kv_row_stride, p.kv_row_stride,
                    min(BKV, kv_len - k0n), tid);
      load_tile<DH>(sV + (buf ^ 1) * TILE_BYTES, vg + (int64_t)k0n * p.kv_row_stride, p.kv_row_stride,
                    min(BKV, kv_len - k0n), tid);
      cp_commit();
      cp_wait<1>();
    } else {
      cp_wait<0>();
    }
    __syncthreads();
    if (j == 0) {
#pragma unroll
      for (int kk = 0; kk < DH / 16; ++kk) {
        const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        ldsm_x4(sQ + tile_off<DH>(row, kk * 2 + (lane >> 4)), qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3]);
      }
    }
    const uint32_t kb = sK + buf * TILE_BYTES, vb = sV + buf * TILE_BYTES;

    // S = Q K^T for this warp's 16 rows x 64 keys
    float s[BKV / 8][4];
#pragma unroll
    for (int nb = 0; nb < BKV / 8; ++nb) { s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk) {
#pragma unroll
      for (int np = 0; np < BKV / 16; ++np) {
        uint32_t b0, b1, b2, b3;
        const int row = np * 16 + (lane & 7) + ((lane >> 4) & 1) * 8;
        ldsm_x4(kb + tile_off<DH>(row, kk * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
        mma_16816(s[np * 2], qf[kk], b0, b1);
        mma_16816(s[np * 2 + 1], qf[kk], b2, b3);
      }
    }

    // scale into the log2 domain, mask the ragged tail, running max
    const int k0 = j * BKV;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nb = 0; nb < BKV / 8; ++nb) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = k0 + nb * 8 + 2 * t + (e & 1);
        float v = s[nb][e] * p.scale_log2;
        if (key >= kv_len) v = -INFINITY;
        s[nb][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    }
    float alpha[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float mn = fmaxf(m_run[r], mx[r]);
      alpha[r] = exp2f(m_run[r] - mn);     // first tile: exp2(-inf) = 0
      m_run[r] = mn;
      l_run[r] *= alpha[r];
    }
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      o[i][0] *= alpha[0]; o[i][1] *= alpha[0];
      o[i][2] *= alpha[1]; o[i][3] *= alpha[1];
    }
    uint32_t pf[BKV / 16][4];
#pragma unroll
    for (int nb = 0; nb < BKV / 8; ++nb) {
      const float p0 = exp2f(s[nb][0] - m_run[0]);
      const float p1 = exp2f(s[nb][1] - m_run[0]);
      const float p2 = exp2f(s[nb][2] - m_run[1]);
      const float p3 = exp2f(s[nb][3] - m_run[1]);
      l_run[0] += p0 + p1;
      l_run[1] += p2 + p3;
      pf[nb >> 1][(nb & 1) * 2 + 0] = pack_bf16(p0, p1);
      pf[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16(p2, p3);
    }

    // O += P V
#pragma unroll
    for (int kk = 0; kk < BKV / 16; ++kk) {
#pragma unroll
      for (int np = 0; np < DH / 16; ++np) {
        uint32_t b0, b1, b2, b3;
        const int row = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        ldsm_x4_t(vb + tile_off<DH>(row, np * 2 + (lane >> 4)), b0, b1, b2, b3);
        mma_16816(o[np * 2], pf[kk], b0, b1);
        mma_16816(o[np * 2 + 1], pf[kk], b2, b3);
      }
    }
    __syncthreads();   // everyone is done with this buffer before the next prefetch overwrites it
  }

#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
  const float inv0 = 1.0f / l_run[0], inv1 = 1.0f / l_run[1];
  const int r0 = warp * 16 + g, r1 = r0 + 8;
  bf16 *og = p.out + (int64_t)(m.row0 + q0) * p.out_stride + h * DH;
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) {
    const int col = i * 8 + 2 * t;
    if (r0 < q_valid)
      *reinterpret_cast<uint32_t *>(og + (int64_t)r0 * p.out_stride + col) = pack_bf16(o[i][0] * inv0, o[i][1] * inv0);
    if (r1 < q_valid)
      *reinterpret_cast<uint32_t *>(og + (int64_t)r1 * p.out_stride + col) = pack_bf16(o[i][2] * inv1, o[i][3] * inv1);
  }
}

template <int DH>
cudaError_t launch(cudaStream_t st, const AttnParams &p, dim3 grid) {
  const int smem = (BQ + 4 * BKV) * DH * 2;
  cudaError_t e = cudaFuncSetAttribute(attention_bf16_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  return launch_kernel(attention_bf16_kernel<DH>, grid, dim3(128), (size_t)smem, st, p);
}

}  // namespace

cudaError_t launch_attention_bf16(cudaStream_t st, const bf16 *q, const bf16 *kc, const bf16 *vc,
                                  const SeqMeta *meta, bf16 *out, int64_t q_stride, int64_t kv_row_stride,
                                  int64_t kv_seq_stride, int64_t out_stride, int n_slots, int max_q_rows,
                                  int H, int dh) {
  AttnParams p;
  p.q = q; p.kc = kc; p.vc = vc; p.out = out; p.meta = meta; p.use_single = 0;
  p.q_stride = q_stride; p.kv_row_stride = kv_row_stride; p.kv_seq_stride = kv_seq_stride; p.out_stride = out_stride;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)dh);
  if (meta == nullptr) {
    // stand-alone call: one sequence, max_q_rows queries, n_slots carries the key count
    p.use_single = 1;
    p.single.seq = 0; p.single.row0 = 0; p.single.n_rows = max_q_rows; p.single.pos0 = 0;
    p.single.kv_len = n_slots; p.single.blk_start = 0; p.single.n_blk_rows = 0; p.single.block = 0;
    n_slots = 1;
  }
  dim3 grid(ceil_div(max_q_rows, BQ), H, n_slots);
  if (dh == 128) return launch<128>(st, p, grid);
  if (dh == 64) return launch<64>(st, p, grid);
  return cudaErrorInvalidValue;
}

}  // namespace l2pd
