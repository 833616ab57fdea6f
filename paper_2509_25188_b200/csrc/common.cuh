// Shared declarations of the l2pd CUDA library (internal).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/l2pd.h"

namespace l2pd {

typedef __nv_bfloat16 bf16;

// One entry per sequence that takes part in the current step (device + pinned host copy).
struct SeqMeta {
  int32_t seq;         // index of the sequence in the batch
  int32_t row0;        // first packed activation row of this sequence
  int32_t n_rows;      // rows computed this step
  int32_t pos0;        // position of row0 (0, or the block start on a cached step)
  int32_t kv_len;      // keys visible to every query of the sequence = L_eff
  int32_t blk_start;   // S_b = P + b*s
  int32_t n_blk_rows;  // min(s, L_eff - S_b): block rows inside L_eff
  int32_t block;       // b
};

// Per-sequence decode state (device arrays of length max_batch).
struct SeqState {
  int32_t *cur_block, *l_eff, *done, *steps, *eot_pos, *forced;
};

// Record the decision kernel writes for the host after each step.
struct StepSummary {
  int32_t block, masks_left, l_eff, done, forced, cur_block;
};

// Device status codes written by kernels whose bounded waits run out.
enum { DEV_OK = 0, DEV_TIMEOUT_PRODUCER = 1, DEV_TIMEOUT_MMA = 2, DEV_TIMEOUT_EPILOGUE = 3 };

inline __host__ __device__ int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline __host__ __device__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

// ---- programmatic dependent launch ------------------------------------------------------------
// Every kernel of the step is launched with programmatic stream serialisation: its blocks may be
// scheduled, and run their set-up, while the previous kernel in the stream is still draining.
// grid_dep_wait() returns once all earlier kernels have completed and their writes are visible;
// every kernel calls it before its first access to global memory that another kernel writes or reads.
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

bool pdl_enabled();   // false when L2PD_NO_PDL=1 (api.cu)

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                 Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- conversions -----------------------------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

// ---- launchers implemented in the .cu files -------------------------------------------------------

// elementwise.cu
template <typename T>
cudaError_t launch_embed_rmsnorm(cudaStream_t st, const int32_t *tokens, int64_t tok_stride,
                                 const SeqMeta *meta, const int32_t *row_slot, const T *emb,
                                 const float *gain, float eps, float *x, T *n, int rows, int d);
// n = RMSNorm(x).  With n_part > 0, first x += part[0] + part[1] + ... (slice s at part + s * part_stride elements,
// added in that order) and x is written back: the fixed-order end of a K-split projection.
template <typename T>
cudaError_t launch_rmsnorm(cudaStream_t st, float *x, const float *gain, float eps, T *n,
                           int rows, int d, const float *part = nullptr, int n_part = 0, int64_t part_stride = 0);
// x += part[0] + part[1] + ... alone (where no RMSNorm follows directly)
cudaError_t launch_add_partials(cudaStream_t st, float *x, const float *part, int n_part, int64_t part_stride, int rows, int d);
template <typename T>
cudaError_t launch_rope_scatter(cudaStream_t st, const T *qkv, const SeqMeta *meta,
                                const int32_t *row_slot, const float2 *cs_table, T *q, T *kc, T *vc,
                                int64_t kv_seq_stride, int rows, int H, int dh);
template <typename T>
cudaError_t launch_final_norm_gather(cudaStream_t st, const float *x, const SeqMeta *meta,
                                     const float *gain, float eps, T *nf, int n_slots, int s,
                                     int rows_padded, int d);
cudaError_t launch_build_row_map(cudaStream_t st, const SeqMeta *meta, int n_slots, int32_t *row_slot, int32_t *row_pos);
// Library-owned copy of a QKV weight [3*H*dh, d] whose q and k rows are reordered inside each head so that the
// rotary pair (i, i + dh/2) sits in adjacent rows (2i, 2i + 1); the v rows are copied as they are.
cudaError_t launch_permute_qkv_rows(cudaStream_t st, const bf16 *src, bf16 *dst, int H, int dh, int d);
cudaError_t launch_state_reset(cudaStream_t st, const int32_t *prompts, int B, int P, int G, int vocab,
                               int mask_id, int32_t *tokens, uint8_t *masked, SeqState s, int32_t *bad);
cudaError_t launch_check_ids(cudaStream_t st, const int32_t *ids, int64_t n, int vocab, int mask_id, int32_t *bad);
cudaError_t launch_gather_response(cudaStream_t st, const int32_t *tokens, int B, int P, int G,
                                   int32_t *out);

// simt.cu : CUDA-core GEMM and attention (fp32 configurations; also a bf16 cross-check path)
enum { EPI_STORE = 0, EPI_RESIDUAL = 1, EPI_SWIGLU = 2, EPI_STORE_F32 = 3, EPI_LMHEAD = 4, EPI_QKV_ROPE = 5 };
template <typename T>
cudaError_t launch_simt_gemm(cudaStream_t st, int epi, const T *A, const T *W, const T *W2, void *C,
                             const float *bias, int M, int N, int K);
template <typename T>
cudaError_t launch_simt_attention(cudaStream_t st, const T *q, const T *kc, const T *vc,
                                  const SeqMeta *meta, const int32_t *row_slot, T *out,
                                  int64_t kv_seq_stride, int rows, int H, int dh, int max_kv);
cudaError_t launch_row_softmax_partials(cudaStream_t st, const float *logits, int R, int V,
                                        float *part_m, float *part_s, int32_t *part_i);

// decide.cu
struct DecideArgs {
  const float *part_m, *part_s;   // [n_tiles, rows_padded]
  const int32_t *part_i;
  int n_tiles, rows_padded;
  const SeqMeta *meta;
  int s, P, G, n_blocks;
  int32_t *tokens; int64_t tok_stride;
  uint8_t *masked;                // [B, G]
  SeqState st;
  const float *w1, *b1, *w2, *b2;
  int n_filter_layers;            // 0: the two-layer filter above; 1..4: fw[k] / fb[k], ReLU between layers (Section 4.4)
  const float *fw[4], *fb[4];
  float tau;
  int use_filter, use_eotp, committed_conf_mode, eot_id;
  int rule;                       // 0 filter (Algorithm 2), 1 fixed confidence threshold, 2 EGP (Section 3.1)
  float conf_threshold;           // rule 1
  const int32_t *ref;             // rule 2: reference answers [B, G]
  float *collect_c; uint8_t *collect_y; int64_t collect_base;   // optional: slot k appends (filter input, pred == ref) as sample collect_base + k
  StepSummary *summary;           // [max_batch], indexed by sequence
  float *o_conf; int32_t *o_pred; float *o_p; uint8_t *o_unmask;   // optional [B, s]
};
cudaError_t launch_decide(cudaStream_t st, const DecideArgs &a, int n_slots);

// filter_train.cu : one AdamW update of the filter on the samples [n0, n0 + n) (Algorithm 1, Eq. 6).
// theta / m / v: packed per layer W_k [s*s], b_k [s] (n_layers of them, 1 .. 4); gpart: [grid, n_layers*(s*s+s) + 1] scratch;
// bc1 / bc2 = 1 - beta^t for this update's step count t; loss_out receives the batch's loss before the update.
struct FilterTrainHyper { float lr, beta1, beta2, eps, weight_decay; };
cudaError_t launch_filter_update(cudaStream_t st, const float *C, const uint8_t *Y, int64_t n0, int64_t n, int s, int n_layers,
                                 float *theta, float *m, float *v, float *gpart, int grid, const FilterTrainHyper &h,
                                 double bc1, double bc2, float *loss_out);

// gemm_tcgen05.cu
struct TmaDesc { CUtensorMap map; };
// Encodes a 2-D bf16 row-major tensor [rows, cols] with a box of [box_rows, 64] and 128-byte swizzle.
l2pd_status make_tma_2d_bf16(TmaDesc *out, const void *ptr, int64_t rows, int64_t cols, int box_rows);
// The same for rows that are `row_stride` elements apart (a multiple of 8).
l2pd_status make_tma_2d_bf16_strided(TmaDesc *out, const void *ptr, int64_t rows, int64_t cols, int64_t row_stride,
                                     int box_rows);
// Output of a GEMM as a 3-D tensor [rows][N / tile_w][tile_w] (bf16, or fp32 for the residual stream) with a
// box of 32 rows x 128 bytes, for the epilogue's staged stores; tile_w = the output columns one tile covers.
l2pd_status make_tma_out_3d(TmaDesc *out, void *ptr, bool fp32, int64_t rows, int64_t N, int tile_w);
// The same for the columns [N - tail_w, N) alone, as one tile of width tail_w (rows are N elements apart).
l2pd_status make_tma_out_tail(TmaDesc *out, void *ptr, bool fp32, int64_t rows, int64_t N, int tail_w);
int lm_head_tile_n(int R, int V, int K, int num_sms);   // tile width of the LM-head GEMM (single CTAs)
// what failed in the calling thread's last context-free call: reported by l2pd_last_error(NULL) (api.cu)
void set_standalone_error(const char *fmt, ...);
// How one GEMM is laid over the SMs: CTAs per tile (1, or 2 = a cta_group::2 pair on a 256-row tile),
// tile width, K slices (residual epilogue only: slices add into X with vector reductions), and row
// slabs per unit (2 = a unit covers two 128 * cta_group row slabs against one load of the weight
// tile, each slab with its own MMA-issuing thread; its accumulators fill tensor memory, so the
// drain is not overlapped with the next unit).
// The B tensor map's box must be tile_n / cta_group rows (SwiGLU: tile_n / 2 for either group size).
// k_interleave = 1 (single CTA, one slab, few rows): the two MMA-issuing threads take alternate k-blocks of the
// unit into two accumulators that the epilogue adds — halves the K loop where instruction issue bounds it
struct GemmPlan { int cta_group, tile_n, k_splits, slabs, k_interleave; };
// max_tile_n caps the tile width (a kernel that chains several projections keeps one ring geometry for all of them)
GemmPlan plan_gemm(int epi, int M, int N, int K, int num_sms, int force_tile_n, int max_k_splits = 4, int max_tile_n = 256);
GemmPlan plan_gemm_pair_one_slab(int epi, int M, int N, int K, int num_sms, int max_k_splits, int max_tile_n);
int effective_k_splits(int K, int k_splits);   // what the launcher makes of a requested K split
struct GemmArgs {
  int epi;                 // EPI_STORE, EPI_RESIDUAL, EPI_SWIGLU, or EPI_LMHEAD
  const TmaDesc *a, *b, *b2;
  const TmaDesc *c;        // output map from make_tma_out_3d (rows = M, tile_w matching tile_n), or null: direct stores
  const TmaDesc *c_tail;   // optional (chained launches): map of the row's last, narrower tile alone, from make_tma_out_tail
  int tail_cols;           // its output columns (a multiple of 16)
  int M, N, K, tile_n;
  int cta_group, k_splits; // 0 / 1 = single CTA, no split
  int slabs;               // 0 / 1 = one row slab per unit, 2 = two
  int k_interleave;        // see GemmPlan
  int a_box_rows;          // 0 / 128: map `a` has a box of 128 rows; M <= 128 only: a box of that many rows (a multiple of 8, >= M)
  void *out;               // bf16 C, fp32 X, or bf16 H
  // LM head
  const float *bias; float *part_m, *part_s; int32_t *part_i; int rows_padded; float *logits;
  int32_t *status;         // device status word
  // EPI_RESIDUAL with k_splits > 1 and part != null: instead of adding into `out`, slice s stores its partial sums
  // at part[(s * part_rows + row) * N + col] (part_rows >= M rounded up to 512, a whole unit of rows; `c`, if given, must map that area);
  // whoever reads X next adds them in slice order (launch_rmsnorm / launch_add_partials): bit-reproducible
  float *part; int part_rows;
  // EPI_QKV_ROPE: columns [0, rope_cols) are rotated in adjacent pairs (2i, 2i + 1) by the angle of pair
  // ((column % dh) / 2) at the row's position; cs_table [dh/2][cs_stride] (cos, sin) indexed [pair][position], row_pos [M]
  int rope_cols, rope_dh, cs_stride; const float2 *cs_table; const int32_t *row_pos;
};
cudaError_t launch_gemm_tcgen05(cudaStream_t st, const GemmArgs &g, int num_sms);
cudaError_t launch_merge_partials(cudaStream_t st, const float *part_m, const float *part_s,
                                  const int32_t *part_i, int n_tiles, int rows_padded, int R,
                                  int32_t *pred, float *conf);

// gemm_chain.cu : several projections (cta_group 2, two row slabs per unit) and the RMSNorms between them in one
// persistent launch; the phases run in the order given, the CTAs meeting at a counter in global memory between them.
struct ChainNorm {        // x += part[0] + part[1] + ... (slice s at part + s * part_stride, in that order), n = RMSNorm(x)
  float *x; const float *gain; float eps; bf16 *n; int rows, d;
  const float *part; int n_part; int64_t part_stride;
};
struct ChainStep { int is_norm; GemmArgs g; ChainNorm nm; };
// CTA pairs of the chain kernel that can be resident at once on the current device (0: the kernel cannot run)
int chain_max_clusters(int num_sms);
bool chain_step_supported(const ChainStep &s);
// A launch runs from a table in device memory: chain_build_table fills the host image (chain_table_bytes() bytes,
// 128-byte aligned) for up to 6 steps holding at most 4 projections, the first step being a projection; the caller
// copies it to the device once and reuses it for every launch of the same steps.  bar: device counter, zero before
// its first use, shared by all tables of a stream; status: device status word.
struct ChainTableInfo { int n_phases, n_stages; size_t smem_bytes; };
size_t chain_table_bytes();
cudaError_t chain_build_table(const ChainStep *steps, int n_steps, unsigned int *bar, int32_t *status, void *h_table,
                              ChainTableInfo *info);
// *bar_base: host copy of the counter's value before this launch, advanced here.  trace: optional device array
// [n_phases][4][2 * n_clusters] of nanosecond stamps (per CTA: phase opened, first and last accumulator ready, phase finished).
cudaError_t launch_gemm_chain(cudaStream_t st, const void *d_table, const ChainTableInfo &info, int n_clusters,
                              unsigned int *bar_base, unsigned long long *trace);

// attention.cu
cudaError_t launch_attention_bf16(cudaStream_t st, const bf16 *q, const bf16 *kc, const bf16 *vc,
                                  const SeqMeta *meta, bf16 *out, int64_t q_stride, int64_t kv_row_stride,
                                  int64_t kv_seq_stride, int64_t out_stride, int n_slots, int max_q_rows,
                                  int H, int dh);


// attention_tc.cu : head size 128 on tcgen05.  tq covers the packed query rows [rows, H*128], tk / tv the
// key / value store as one matrix of rows (layer, sequence, position) x H*128; all with a box of 128 rows.
// kv_packed != 0: keys and values lie in the packed activation rows instead (row = the sequence's row0 + key).
bool attention_tc_supported(int dh, int64_t q_stride, int64_t kv_row_stride, int64_t out_stride);
cudaError_t launch_attention_tc(cudaStream_t st, const TmaDesc &tq, const TmaDesc &tk, const TmaDesc &tv,
                                const SeqMeta *meta, bf16 *out, int64_t out_stride, int kv_rows_per_seq,
                                int kv_row_base, int kv_packed, int n_slots, int max_q_rows, int H, int32_t *status);

}  // namespace l2pd
