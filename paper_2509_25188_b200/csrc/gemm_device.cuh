// Device-side pieces shared by the tcgen05 GEMM kernels: tile constants, the per-launch parameter
// block, and the epilogues that drain an accumulator from tensor memory (direct stores, or staged
// through shared memory and written by the TMA unit).
#pragma once
#include <math.h>

#include "common.cuh"
#include "ptx.cuh"

namespace l2pd {
namespace gemm_dev {

constexpr int TILE_M = 128;
constexpr int TILE_K = 64;                       // 64 bf16 = 128 bytes = one swizzle row
constexpr int A_STAGE_BYTES = TILE_M * TILE_K * 2;
constexpr int MAX_STAGES = 8;
constexpr int TMEM_COLS = 512;
constexpr int ACC_COLS = 256;                    // columns per accumulator buffer
constexpr int SMEM_BUDGET = 227 * 1024;

struct KParams {
  int M, N, K, tile_n, n_stages, b_stage_bytes;
  int slabs, a_stage_bytes;         // row slabs (of 128 * CG rows) one unit covers: 1, or 2 = accumulators not double-buffered
  int m_tiles, n_tiles, k_splits;   // m_tiles counts row tiles of 128 * CG * slabs rows
  int group_m;                      // row tiles per raster group (see the unit order in gemm_body)
  void *out;
  const float *bias;
  float *part_m, *part_s;
  int32_t *part_i;
  int rows_padded;
  float *logits;
  int32_t *status;
  int out_tma;          // 1: the epilogue may stage its output in shared memory and store it through tmC
  int out_full_tiles;   // column tiles that lie wholly inside the row (the others use direct stores)
  int out_tail_cols;    // > 0: the last, narrower tile has its own output map and is staged too (that many output columns)
  int gate;             // 1: every unit's epilogue is staged; the producer keeps off the staging area meanwhile
  float *part; int part_rows;      // EPI_RESIDUAL with K slices: slice s stores its partial sums at part[s * part_rows + row][N]
  int rope_cols, rope_dh, cs_stride;   // EPI_QKV_ROPE, see GemmArgs
  const float2 *cs_table;
  const int32_t *row_pos;
  int kil;   // 1: the unit's k-blocks alternate between the two MMA issuers (accumulators 0 and 1, added in the epilogue)
  // Few rows (M <= 128, one row tile): an activation load brings only a_box_bytes = (M rounded up to 8) x 128 bytes
  // instead of a whole 128-row tile; the MMA still reads 128 rows, the rest being whatever shared memory holds, into
  // accumulator rows that are never stored.  a_peer_loads = 0: the second CTA of a pair has no rows and loads none.
  int a_box_bytes, a_peer_loads;
};

__device__ __forceinline__ void fail(int32_t *status, int code) {
  if (status) atomicCAS(status, 0, code);
}

// silu(g) * u with the fast exponential and division (a few ulp, far below the bf16 rounding of the result)
__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

// Emitters: what the epilogue does with 16 consecutive accumulator columns of one row.
// `valid` = columns left in the row from the first of the 16 (the row length is a multiple of 8).
__device__ __forceinline__ void emit_store16(bf16 *dst, const uint32_t *v, int valid) {   // 16 fp32 -> 16 bf16, 32 bytes
#pragma unroll
  for (int hseg = 0; hseg < 2; ++hseg) {
    if (hseg * 8 >= valid) break;
    uint4 pk;
    uint32_t *pw = reinterpret_cast<uint32_t *>(&pk);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 t = __floats2bfloat162_rn(__uint_as_float(v[hseg * 8 + 2 * i]), __uint_as_float(v[hseg * 8 + 2 * i + 1]));
      pw[i] = *reinterpret_cast<uint32_t *>(&t);
    }
    *reinterpret_cast<uint4 *>(dst + hseg * 8) = pk;
  }
}
// mode 0: x += acc (read-modify-write), 1: atomic x += acc, 2: plain store (a K slice's partial sums)
__device__ __forceinline__ void emit_residual16(float *px, const uint32_t *v, int mode, int valid) {
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    if (g * 4 >= valid) break;
    if (mode == 2) {
      *reinterpret_cast<float4 *>(px + 4 * g) = make_float4(__uint_as_float(v[4 * g + 0]), __uint_as_float(v[4 * g + 1]),
                                                            __uint_as_float(v[4 * g + 2]), __uint_as_float(v[4 * g + 3]));
    } else if (mode == 1) {
      ptx::red_add_v4(px + 4 * g, __uint_as_float(v[4 * g + 0]), __uint_as_float(v[4 * g + 1]),
                      __uint_as_float(v[4 * g + 2]), __uint_as_float(v[4 * g + 3]));
    } else {
      float4 x = *reinterpret_cast<float4 *>(px + 4 * g);
      x.x += __uint_as_float(v[4 * g + 0]);
      x.y += __uint_as_float(v[4 * g + 1]);
      x.z += __uint_as_float(v[4 * g + 2]);
      x.w += __uint_as_float(v[4 * g + 3]);
      *reinterpret_cast<float4 *>(px + 4 * g) = x;
    }
  }
}
__device__ __forceinline__ void emit_swiglu16(bf16 *dst, const uint32_t *g, const uint32_t *u, int valid) {
#pragma unroll
  for (int hseg = 0; hseg < 2; ++hseg) {
    if (hseg * 8 >= valid) break;
    uint4 pk;
    uint32_t *pw = reinterpret_cast<uint32_t *>(&pk);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float g0 = __uint_as_float(g[hseg * 8 + 2 * i]), g1 = __uint_as_float(g[hseg * 8 + 2 * i + 1]);
      const float u0 = __uint_as_float(u[hseg * 8 + 2 * i]), u1 = __uint_as_float(u[hseg * 8 + 2 * i + 1]);
      __nv_bfloat162 t = __floats2bfloat162_rn(silu_mul(g0, u0), silu_mul(g1, u1));
      pw[i] = *reinterpret_cast<uint32_t *>(&t);
    }
    *reinterpret_cast<uint4 *>(dst + hseg * 8) = pk;
  }
}

// Rotary embedding on 32 (or 16) consecutive accumulator columns of one row, starting at the even column col0:
// the pair (x1, x2) = columns (2t, 2t + 1) becomes (x1 cos - x2 sin, x2 cos + x1 sin), the angle being that of
// pair index ((column % dh) / 2) at position pos.  Columns from rope_cols on (the v part) are left alone.
struct RopeArgs { int rope_cols, rope_dh, cs_stride; const float2 *cs_table; };   // by value: lives in registers
// The angles of the 16 pairs starting at column col0 for the row at position pos.  The table is laid out
// [pair][position]: the 32 rows of a warp are consecutive positions, so a load is one line.
__device__ __forceinline__ void rope_fetch(const RopeArgs &r, float2 (&a)[16], int col0, int pos) {
  if (col0 >= r.rope_cols) return;               // a chunk of v columns (warp-uniform)
  const float2 *cs = r.cs_table + pos;
  const int mask = r.rope_dh - 1;
#pragma unroll
  for (int t = 0; t < 16; ++t) a[t] = __ldg(cs + (int64_t)(((col0 + 2 * t) & mask) >> 1) * r.cs_stride);
}
__device__ __forceinline__ void rope_apply(const RopeArgs &r, uint32_t (&v)[32], const float2 (&a)[16], int col0, int ncols) {
  if (col0 >= r.rope_cols) return;
#pragma unroll
  for (int t = 0; t < 16; ++t) {
    if (2 * t < ncols && col0 + 2 * t < r.rope_cols) {
      const float x1 = __uint_as_float(v[2 * t]), x2 = __uint_as_float(v[2 * t + 1]);
      v[2 * t] = __float_as_uint(x1 * a[t].x - x2 * a[t].y);
      v[2 * t + 1] = __float_as_uint(x2 * a[t].x + x1 * a[t].y);
    }
  }
}
// The same for 8 pairs (16 columns).
__device__ __forceinline__ void rope_fetch8(const RopeArgs &r, float2 (&a)[8], int col0, int pos) {
  if (col0 >= r.rope_cols) return;
  const float2 *cs = r.cs_table + pos;
  const int mask = r.rope_dh - 1;
#pragma unroll
  for (int t = 0; t < 8; ++t) a[t] = __ldg(cs + (int64_t)(((col0 + 2 * t) & mask) >> 1) * r.cs_stride);
}
__device__ __forceinline__ void rope_pairs(const RopeArgs &r, uint32_t (&v)[32], int col0, int ncols, int pos) {
  if (col0 >= r.rope_cols) return;
  float2 a[16];
  rope_fetch(r, a, col0, pos);                   // all 16 angles are fetched before any is used
  rope_apply(r, v, a, col0, ncols);
}

// Drains one 128-row x tile_n accumulator from tensor memory (this warp's 32 lanes) and applies the
// epilogue with per-thread stores (a thread owns one row).  The loads run one step ahead of the
// arithmetic and stores: while chunk c is converted and written, chunk c + 1 is in flight
// (tcgen05.wait::ld covers every load issued so far).
// K slices of the residual epilogue either add into X (`res_mode` 1) or store their partial sums to
// `res_base`, the slice's own [rows][N] area (`res_mode` 2), for a later fixed-order sum.
template <int EPI>
// two_acc: the unit's sum is spread over two accumulators (ACC_COLS columns apart), added here.
__device__ __forceinline__ void drain_tile(const KParams &p, uint32_t taddr, int row, int nt, int res_mode, float *res_base,
                                           bool two_acc = false) {
  const bool row_ok = row < p.M;
  const int half_n = p.tile_n >> 1;
  if (EPI == EPI_STORE || EPI == EPI_RESIDUAL || EPI == EPI_QKV_ROPE) {
    const int pos = (EPI == EPI_QKV_ROPE && row_ok) ? p.row_pos[row] : 0;
    const RopeArgs rope{p.rope_cols, p.rope_dh, p.cs_stride, p.cs_table};
    // 32 columns per step (tile_n is a multiple of 16: the last step may hold 16)
    const int n0 = nt * p.tile_n, n = p.tile_n;
    uint32_t va[32], vb[32];
    auto load = [&](uint32_t (&v)[32], int c) {
      if (n - c >= 32) ptx::tmem_ld_x32(taddr + c, v);
      else ptx::tmem_ld_x16(taddr + c, v);
    };
    auto emit = [&](uint32_t (&v)[32], int c) {
      if (!row_ok) return;
      if (EPI == EPI_QKV_ROPE) rope_pairs(rope, v, n0 + c, min(32, n - c), pos);
#pragma unroll
      for (int h16 = 0; h16 < 2; ++h16) {
        const int col = n0 + c + 16 * h16;
        if (c + 16 * h16 < n && col < p.N) {
          if (EPI != EPI_RESIDUAL) emit_store16(reinterpret_cast<bf16 *>(p.out) + (int64_t)row * p.N + col, v + 16 * h16, p.N - col);
          else emit_residual16(res_base + (int64_t)row * p.N + col, v + 16 * h16, res_mode, p.N - col);
        }
      }
    };
    if (two_acc) {
      for (int c = 0; c < n; c += 32) {
        load(va, c);
        if (n - c >= 32) ptx::tmem_ld_x32(taddr + ACC_COLS + c, vb);
        else ptx::tmem_ld_x16(taddr + ACC_COLS + c, vb);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) va[i] = __float_as_uint(__uint_as_float(va[i]) + __uint_as_float(vb[i]));
        emit(va, c);
      }
      return;
    }
    load(va, 0);
    for (int c = 0; c < n; c += 64) {
      ptx::tmem_ld_wait();
      if (c + 32 < n) load(vb, c + 32);
      emit(va, c);
      if (c + 32 >= n) break;
      ptx::tmem_ld_wait();
      if (c + 64 < n) load(va, c + 64);
      emit(vb, c + 32);
    }
  } else if (EPI == EPI_SWIGLU) {
    bf16 *H = reinterpret_cast<bf16 *>(p.out);
    const int n0 = nt * half_n;
    uint32_t ga[16], ua[16], gb[16], ub[16];
    auto load = [&](uint32_t *g, uint32_t *u, int c) {
      ptx::tmem_ld_x16(taddr + c, g);
      ptx::tmem_ld_x16(taddr + half_n + c, u);
    };
    auto emit = [&](const uint32_t *g, const uint32_t *u, int c) {
      if (row_ok && n0 + c < p.N) emit_swiglu16(H + (int64_t)row * p.N + n0 + c, g, u, min(p.N - n0 - c, half_n - c));
    };
    if (two_acc) {
      for (int c = 0; c < half_n; c += 16) {
        load(ga, ua, c);
        ptx::tmem_ld_x16(taddr + ACC_COLS + c, gb);
        ptx::tmem_ld_x16(taddr + ACC_COLS + half_n + c, ub);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          ga[i] = __float_as_uint(__uint_as_float(ga[i]) + __uint_as_float(gb[i]));
          ua[i] = __float_as_uint(__uint_as_float(ua[i]) + __uint_as_float(ub[i]));
        }
        emit(ga, ua, c);
      }
      return;
    }
    load(ga, ua, 0);
    for (int c = 0; c < half_n; c += 32) {
      ptx::tmem_ld_wait();
      if (c + 16 < half_n) load(gb, ub, c + 16);
      emit(ga, ua, c);
      if (c + 16 >= half_n) break;
      ptx::tmem_ld_wait();
      if (c + 32 < half_n) load(ga, ua, c + 32);
      emit(gb, ub, c + 16);
    }
  } else {  // EPI_LMHEAD
    uint32_t v[16];
    const float L2E = 1.4426950408889634f;
    const int n0 = nt * p.tile_n;
    float m_run = -INFINITY, s_run = 0.f;
    int i_run = 0x7fffffff;
    for (int c = 0; c < p.tile_n; c += 16) {
      ptx::tmem_ld_x16(taddr + c, v);
      ptx::tmem_ld_wait();
      if (row_ok && n0 + c < p.N) {
        float f[16];
        float cm = -INFINITY;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int col = n0 + c + i;
          float val = __uint_as_float(v[i]);
          if (col < p.N) { if (p.bias) val += __ldg(p.bias + col); }
          else val = -INFINITY;
          f[i] = val;
          cm = fmaxf(cm, val);
        }
        if (p.logits) {
#pragma unroll
          for (int i = 0; i < 16; ++i)
            if (n0 + c + i < p.N) p.logits[(int64_t)row * p.N + n0 + c + i] = f[i];
        }
        if (cm > m_run) {
          s_run *= exp2f((m_run - cm) * L2E);
          m_run = cm;
          int ci = 0;
#pragma unroll
          for (int i = 15; i >= 0; --i) if (f[i] == cm) ci = i;   // lowest index holding the max
          i_run = n0 + c + ci;
        }
        float add = 0.f;
#pragma unroll
        for (int i = 0; i < 16; ++i) add += exp2f((f[i] - m_run) * L2E);
        s_run += add;
      }
    }
    if (row_ok) {
      const int64_t o = (int64_t)nt * p.rows_padded + row;
      p.part_m[o] = m_run;
      p.part_s[o] = s_run;
      p.part_i[o] = i_run;
    }
  }
}

// The same through shared memory and TMA: a thread owns one accumulator row, so direct stores touch
// 32 different lines per instruction; instead each warp lays 128 bytes of 32 rows into a swizzled
// staging tile (4 KB) and one thread hands it to the TMA unit, which writes whole lines (bf16
// outputs) or adds them into X in L2 (fp32 residual).  The output tensor map is 3-D
// [rows][column tile][column in tile], so a box that runs past the tile's width is clipped there,
// and rows beyond M are clipped by the map's row count.
// The warp's STAGE_BUFS staging tiles lie over the A operands of the ring's last two stages and are
// used in turn.  That memory is idle during a CTA's last unit; for earlier units (two-slab units,
// whose drain is not overlapped anyway) the producer refills those two stages only after the
// epilogue warps have reported the staging area free.
// Everything below is written as force-inlined functions over arrays passed by reference (not lambdas
// over pointers): the accumulator chunks and the angles then stay in registers in every instantiation.
constexpr int STAGE_BUFS = 2;

struct StagedOut {
  const CUtensorMap *tmC;
  uint32_t stage0, stage, sw;
  int lane, n_flush, map_nt, row0;
  bool add;                      // fp32 residual added into X by the TMA unit (no K slices' partial sums)
  __device__ __forceinline__ StagedOut(const CUtensorMap *m, uint32_t s0, int ln, int mnt, int r0, bool add_)
      : tmC(m), stage0(s0), stage(s0), sw((uint32_t)(ln & 7)), lane(ln), n_flush(0), map_nt(mnt), row0(r0), add(add_) {}
  __device__ __forceinline__ uint32_t chunk_addr(int ch) const { return stage + lane * 128 + (((uint32_t)ch ^ sw) << 4); }
  __device__ __forceinline__ void st16(int ch, uint32_t a, uint32_t b, uint32_t c, uint32_t d) const {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(chunk_addr(ch)), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
  }
  // hand the staged 32 x 128-byte tile (columns from c0 on) to the TMA unit
  __device__ __forceinline__ void flush(int c0) {
    ptx::fence_proxy_async();
    __syncwarp();
    if (lane == 0) {
      if (add) ptx::tma_reduce_add_3d(tmC, stage, c0, map_nt, row0);
      else ptx::tma_store_3d(tmC, stage, c0, map_nt, row0);
      ptx::bulk_commit();
    }
    ++n_flush;
  }
  // pick the next staging tile; the flush that used it STAGE_BUFS turns ago has read it
  __device__ __forceinline__ void reuse() {
    stage = stage0 + (uint32_t)(n_flush % STAGE_BUFS) * 4096u;
    if (n_flush >= STAGE_BUFS) {
      if (lane == 0) ptx::bulk_wait_read_n<STAGE_BUFS - 1>();
      __syncwarp();
    }
  }
};

__device__ __forceinline__ uint32_t pack_bf16x2(uint32_t a, uint32_t b) {
  __nv_bfloat162 t = __floats2bfloat162_rn(__uint_as_float(a), __uint_as_float(b));
  return *reinterpret_cast<uint32_t *>(&t);
}
__device__ __forceinline__ void tmem_load_cols(uint32_t taddr, uint32_t (&v)[32], int cols_left) {
  if (cols_left >= 32) ptx::tmem_ld_x32(taddr, v);
  else ptx::tmem_ld_x16(taddr, v);
}
// 32 accumulator columns starting at column c of the tile (the upper 16 may lie beyond it): rotation, conversion,
// staging, and the hand-over once a staging tile is full or the tile ends
template <int EPI>
__device__ __forceinline__ void emit_cols(StagedOut &o, const uint32_t (&v)[32], int c, int n) {
  if (EPI == EPI_RESIDUAL) {
    o.reuse();
#pragma unroll
    for (int ch = 0; ch < 8; ++ch) o.st16(ch, v[4 * ch], v[4 * ch + 1], v[4 * ch + 2], v[4 * ch + 3]);
    o.flush(c);
  } else {
    const int hb = (c >> 5) & 1;              // which 64-byte half of the 128-byte staging row
    if (hb == 0) o.reuse();
#pragma unroll
    for (int ch = 0; ch < 4; ++ch)
      o.st16(hb * 4 + ch, pack_bf16x2(v[8 * ch], v[8 * ch + 1]), pack_bf16x2(v[8 * ch + 2], v[8 * ch + 3]),
             pack_bf16x2(v[8 * ch + 4], v[8 * ch + 5]), pack_bf16x2(v[8 * ch + 6], v[8 * ch + 7]));
    if (hb == 1 || c + 32 >= n) o.flush(c & ~63);
  }
}
// 16 accumulator columns starting at column c of the tile, rotated: the pair (x1, x2) = columns (2t, 2t + 1) becomes
// (x1 cos - x2 sin, x2 cos + x1 sin); columns from rope_cols on (the v part) are copied.  32 bytes of the staging row.
__device__ __forceinline__ void emit_rope_cols(StagedOut &o, const RopeArgs &rope, const uint32_t (&v)[16], const float2 (&a)[8], int c,
                                               int n, int col_base) {
  const bool rot = col_base + c < rope.rope_cols;   // warp-uniform
  uint32_t pk[8];
#pragma unroll
  for (int t = 0; t < 8; ++t) {
    const float x1 = __uint_as_float(v[2 * t]), x2 = __uint_as_float(v[2 * t + 1]);
    const bool on = rot && col_base + c + 2 * t < rope.rope_cols;
    const float cs = on ? a[t].x : 1.0f, sn = on ? a[t].y : 0.0f;
    __nv_bfloat162 h2 = __floats2bfloat162_rn(x1 * cs - x2 * sn, x2 * cs + x1 * sn);
    pk[t] = *reinterpret_cast<uint32_t *>(&h2);
  }
  const int qb = (c >> 4) & 3;                // which 32-byte quarter of the staging row
  if (qb == 0) o.reuse();
  o.st16(qb * 2, pk[0], pk[1], pk[2], pk[3]);
  o.st16(qb * 2 + 1, pk[4], pk[5], pk[6], pk[7]);
  if (qb == 3 || c + 16 >= n) o.flush(c & ~63);
}
// SwiGLU: 16 gate + 16 up columns give 16 outputs = 32 bytes of the staging row
__device__ __forceinline__ void emit_swiglu_cols(StagedOut &o, const uint32_t (&g)[16], const uint32_t (&u)[16], int c, int hn) {
  const int qb = (c >> 4) & 3;                // which 32-byte quarter of the staging row
  if (qb == 0) o.reuse();
#pragma unroll
  for (int hseg = 0; hseg < 2; ++hseg) {
    uint32_t pw[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float g0 = __uint_as_float(g[hseg * 8 + 2 * i]), g1 = __uint_as_float(g[hseg * 8 + 2 * i + 1]);
      const float u0 = __uint_as_float(u[hseg * 8 + 2 * i]), u1 = __uint_as_float(u[hseg * 8 + 2 * i + 1]);
      __nv_bfloat162 t = __floats2bfloat162_rn(silu_mul(g0, u0), silu_mul(g1, u1));
      pw[i] = *reinterpret_cast<uint32_t *>(&t);
    }
    o.st16(qb * 2 + hseg, pw[0], pw[1], pw[2], pw[3]);
  }
  if (qb == 3 || c + 16 >= hn) o.flush(c & ~63);
}

// tail_cols > 0: the row's last, narrower column tile — only its first tail_cols output columns are drained, and tmC
// is a map of that tile alone (tile coordinate 0, inner extent tail_cols), so boxes are clipped at the row's end.
// two_acc: the unit's sum is spread over two accumulators ACC_COLS columns apart (two MMA issuers on alternate
// k-blocks); they are added here, first + second, before the epilogue (not for the rotating epilogue).
template <int EPI>
__device__ __forceinline__ void drain_tile_staged(const KParams &p, const CUtensorMap *tmC, uint32_t taddr, int row0,
                                                  int nt, uint32_t stage0, int lane, bool res_store, int tail_cols = 0,
                                                  bool two_acc = false) {
  const int half_n = p.tile_n >> 1;
  StagedOut o(tmC, stage0, lane, tail_cols > 0 ? 0 : nt, row0, EPI == EPI_RESIDUAL && !res_store);
  if (EPI == EPI_QKV_ROPE) {
    // 16 columns at a time; the angles of a chunk are requested together with its accumulator columns, one chunk
    // ahead of their use
    const int n = tail_cols > 0 ? tail_cols : p.tile_n;
    const int col_base = nt * p.tile_n;
    const int pos = row0 + lane < p.M ? p.row_pos[row0 + lane] : 0;
    const RopeArgs rope{p.rope_cols, p.rope_dh, p.cs_stride, p.cs_table};
    uint32_t va[16], vb[16];
    float2 aa[8], ab[8];
    ptx::tmem_ld_x16(taddr, va);
    rope_fetch8(rope, aa, col_base, pos);
    for (int c = 0; c < n; c += 32) {
      ptx::tmem_ld_wait();
      if (c + 16 < n) { ptx::tmem_ld_x16(taddr + c + 16, vb); rope_fetch8(rope, ab, col_base + c + 16, pos); }
      emit_rope_cols(o, rope, va, aa, c, n, col_base);
      if (c + 16 >= n) break;
      ptx::tmem_ld_wait();
      if (c + 32 < n) { ptx::tmem_ld_x16(taddr + c + 32, va); rope_fetch8(rope, aa, col_base + c + 32, pos); }
      emit_rope_cols(o, rope, vb, ab, c + 16, n, col_base);
    }
  } else if (EPI == EPI_STORE || EPI == EPI_RESIDUAL) {
    const int n = tail_cols > 0 ? tail_cols : p.tile_n;
    uint32_t va[32], vb[32];
    if (two_acc) {
      for (int c = 0; c < n; c += 32) {
        tmem_load_cols(taddr + c, va, n - c);
        tmem_load_cols(taddr + ACC_COLS + c, vb, n - c);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) va[i] = __float_as_uint(__uint_as_float(va[i]) + __uint_as_float(vb[i]));
        emit_cols<EPI>(o, va, c, n);
      }
      return;
    }
    tmem_load_cols(taddr, va, n);
    for (int c = 0; c < n; c += 64) {
      ptx::tmem_ld_wait();
      if (c + 32 < n) tmem_load_cols(taddr + c + 32, vb, n - c - 32);
      emit_cols<EPI>(o, va, c, n);
      if (c + 32 >= n) break;
      ptx::tmem_ld_wait();
      if (c + 64 < n) tmem_load_cols(taddr + c + 64, va, n - c - 64);
      emit_cols<EPI>(o, vb, c + 32, n);
    }
  } else {   // EPI_SWIGLU
    const int hn = tail_cols > 0 ? tail_cols : half_n;   // output columns to drain
    uint32_t ga[16], ua[16], gb[16], ub[16];
    if (two_acc) {
      for (int c = 0; c < hn; c += 16) {
        ptx::tmem_ld_x16(taddr + c, ga);
        ptx::tmem_ld_x16(taddr + half_n + c, ua);
        ptx::tmem_ld_x16(taddr + ACC_COLS + c, gb);
        ptx::tmem_ld_x16(taddr + ACC_COLS + half_n + c, ub);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          ga[i] = __float_as_uint(__uint_as_float(ga[i]) + __uint_as_float(gb[i]));
          ua[i] = __float_as_uint(__uint_as_float(ua[i]) + __uint_as_float(ub[i]));
        }
        emit_swiglu_cols(o, ga, ua, c, hn);
      }
      return;
    }
    ptx::tmem_ld_x16(taddr, ga);
    ptx::tmem_ld_x16(taddr + half_n, ua);
    for (int c = 0; c < hn; c += 32) {
      ptx::tmem_ld_wait();
      if (c + 16 < hn) { ptx::tmem_ld_x16(taddr + c + 16, gb); ptx::tmem_ld_x16(taddr + half_n + c + 16, ub); }
      emit_swiglu_cols(o, ga, ua, c, hn);
      if (c + 16 >= hn) break;
      ptx::tmem_ld_wait();
      if (c + 32 < hn) { ptx::tmem_ld_x16(taddr + c + 32, ga); ptx::tmem_ld_x16(taddr + half_n + c + 32, ua); }
      emit_swiglu_cols(o, gb, ub, c + 16, hn);
    }
  }
}

}  // namespace gemm_dev

// Fills the kernel's parameter block for one GEMM (gemm_tcgen05.cu).  stages / b_stage_bytes = 0: the deepest
// ring the shared memory holds for this tile; otherwise the given ring geometry.
cudaError_t fill_kparams(const GemmArgs &g, int stages, int b_stage_bytes, gemm_dev::KParams &p, bool chained = false);

}  // namespace l2pd
