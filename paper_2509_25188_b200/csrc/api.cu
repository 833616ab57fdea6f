// C ABI of the l2pd library: context, decode state, one denoising step, the decode loop.
// Host code only orchestrates; every arithmetic step of the path runs in the kernels of the
// other files.  Nothing here falls back to the CPU: a failed CUDA call is an error status.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"

using namespace l2pd;

struct l2pd_ctx {
  l2pd_config cfg;
  int device = 0, num_sms = 148;
  bool force_simt = false;   // L2PD_FORCE_SIMT=1: bf16 GEMMs and attention on the CUDA-core cross-check kernels
  bool attn_tc = false;      // head size 128: attention on tcgen05 (L2PD_ATTN_WARP=1 keeps the mma.sync kernel)
  // RoPE in the QKV epilogue (tcgen05 attention, no prefix cache; L2PD_NO_ROPE_FUSION=1 turns it off): the context
  // owns copies of the QKV weights with the q / k rows of each head reordered so that rotary pairs are adjacent;
  // q and k then live in that order, which leaves every q . k unchanged; attention reads q, k, v from the packed qkv rows
  bool fuse_rope = false;
  std::vector<void *> wqkv_perm;
  int32_t *d_row_pos = nullptr;
  TmaDesc tq_packed, tk_packed, tv_packed;

  // weights (borrowed device pointers)
  const void *tok_emb = nullptr, *lm_head = nullptr;
  std::vector<const void *> wqkv, wo, w_gate, w_up, w_down;
  std::vector<const float *> norm1, norm2;
  const float *final_norm = nullptr, *lm_bias = nullptr, *fw1 = nullptr, *fb1 = nullptr, *fw2 = nullptr, *fb2 = nullptr;

  // decode state
  int B = 0, P = 0, G = 0;
  int rule = L2PD_RULE_FILTER;          // test applied to masked positions (l2pd_set_unmask_rule)
  float conf_threshold = 0.9f;
  const int32_t *d_ref = nullptr;       // EGP: reference answers [ref_rows, ref_len], borrowed
  int ref_rows = 0, ref_len = 0;
  int n_filter_layers = 0;              // l2pd_set_filter: 0 = the two-layer filter given at init
  const float *flt_w[4] = {}, *flt_b[4] = {};
  float *collect_c = nullptr;           // sample sink of l2pd_set_collect
  uint8_t *collect_y = nullptr;
  int64_t collect_cap = 0, collect_n = 0;
  bool has_state = false;
  int32_t *d_tokens = nullptr;
  uint8_t *d_masked = nullptr;
  int32_t *d_state_ints = nullptr;   // 6 arrays of max_batch
  SeqState st{};
  std::vector<int> h_cur_block, h_l_eff, h_done, h_steps, h_cache_block;
  int n_active = 0;
  int total_steps = 0;

  // workspace
  int64_t max_rows = 0;              // capacity in activation rows (multiple of 128)
  int64_t max_lm_rows = 0;           // max_batch * s rounded up to 128
  float *x = nullptr;
  void *n = nullptr, *qkv = nullptr, *q = nullptr, *att = nullptr, *h = nullptr, *nf = nullptr;
  void *kc = nullptr, *vc = nullptr;
  int64_t kv_seq_stride = 0, kv_layer_stride = 0;
  float *part = nullptr;             // part_m | part_s | part_i
  int64_t part_tiles_cap = 0;
  float *logits_f32 = nullptr;       // fp32 configurations: [max_lm_rows, V]
  SeqMeta *d_meta = nullptr, *h_meta = nullptr;
  int32_t *d_row_slot = nullptr;
  StepSummary *d_summary = nullptr, *h_summary = nullptr;
  int32_t *d_status = nullptr, *h_status = nullptr;
  float2 *cs_table = nullptr;
  // partial sums of the K slices of the O and down projections, [4][ksum_rows][d] fp32: summed in slice order by the
  // RMSNorm that follows (bit-reproducible, unlike additions into x in completion order)
  float *ksum = nullptr;
  int64_t ksum_rows = 0;
  float2 *cs_table_t = nullptr;      // the same table as [pair][position] (fused rotation in the QKV epilogue)

  // TMA descriptors (bf16 path)
  TmaDesc ta_n, ta_att, ta_h, ta_nf, ta_q, t_kstore, t_vstore;
  // steps of at most 128 rows load only their rows: the same maps with a box of `a_box` rows (a_box_nf for the LM head's)
  TmaDesc ta_n_s, ta_att_s, ta_h_s, ta_nf_s;
  int a_box = 0, a_box_nf = 0;
  // output maps of the four projections (staged epilogue stores); re-encoded when rows or tile width change
  TmaDesc tc_qkv, tc_o, tc_h, tc_down;
  // the same for each projection's last, narrower column tile (chained launches stage every tile); tail width, 0 = none
  TmaDesc tct_qkv, tct_o, tct_h, tct_down;
  int tail_qkv = 0, tail_o = 0, tail_h = 0, tail_down = 0;
  int tc_rows = -1, tcw_qkv = 0, tcw_o = 0, tcw_h = 0, tcw_down = 0;   // tile width encoded (0 = none, -w = not usable for w)
  std::vector<TmaDesc> tb_qkv, tb_o, tb_gate, tb_up, tb_down;
  TmaDesc tb_lm;
  GemmPlan pl_qkv{}, pl_o{}, pl_gu{}, pl_down{};
  int box_qkv = 0, box_o = 0, box_gu = 0, box_down = 0, tn_lm = 0;

  // several projections per launch (gemm_chain.cu): on when every projection of the step runs on SM pairs with
  // two row slabs per unit and K slices store partial sums
  int chain_mode = 0;                // l2pd_set_chain: 0 one launch per projection, 1 chained launches, 2 the chained form's tiling in single launches
  int chain_clusters = 0;            // CTA pairs that can be resident at once (0: kernel not usable here)
  unsigned int *d_chain_bar = nullptr;
  unsigned int chain_bar_base = 0;   // host copy of the counter's value
  // one table per chained launch of a step (first QKV, then one per layer), device-resident, rebuilt when the step's
  // row count (hence tiling and output maps) changes
  uint8_t *d_chain_tabs = nullptr, *h_chain_tabs = nullptr;
  std::vector<ChainTableInfo> chain_info;
  int chain_tab_rows = -1;
  unsigned long long *d_chain_trace = nullptr;   // l2pd_chain_trace_enable: [launch][phase][4][CTA] stamps of the last step
  int64_t chain_trace_cap = 0;
  int chain_trace_launches = 0, chain_trace_phases = 0, chain_trace_ctas = 0;

  // debug capture
  float *cap = nullptr;
  int64_t cap_stride = 0;
  int last_rows = 0;

  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  float last_ms = -1.f;

  // per-kernel timing (CUDA events around the launches of the selected kinds)
  uint32_t prof_mask = 0;
  std::vector<cudaEvent_t> prof_events;          // pairs: begin, end
  std::vector<int> prof_pending_kind;            // kind of each recorded pair of the current step
  double prof_ms[L2PD_K_COUNT] = {};
  int64_t prof_launches[L2PD_K_COUNT] = {};
  int64_t launches = 0;
  std::string err;
};

namespace l2pd {
bool pdl_enabled() {
  static const bool on = [] { const char *e = getenv("L2PD_NO_PDL"); return !(e && e[0] == '1'); }();
  return on;
}
}  // namespace l2pd

namespace {

constexpr int CHAIN_TILE_N = 176;       // widest tile of a step that chains projections
constexpr int CHAIN_MAX_ROWS = 1536;    // steps of more rows run one launch per projection (the launch is then a small part)
constexpr int CHAIN_TRACE_STAMPS = 4;   // stamps per phase and CTA
constexpr int CHAIN_TRACE_PHASES = 6;   // phases a chained launch can hold (slots per launch in the trace)

l2pd_status set_err(l2pd_ctx *c, l2pd_status s, const char *fmt, ...) {
  if (c) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    c->err = buf;
  }
  return s;
}

#define CK(call)                                                                                   \
  do {                                                                                             \
    cudaError_t e_ = (call);                                                                       \
    if (e_ != cudaSuccess)                                                                         \
      return set_err(c, e_ == cudaErrorMemoryAllocation ? L2PD_ERR_OOM : L2PD_ERR_CUDA, "%s: %s", \
                     #call, cudaGetErrorString(e_));                                               \
  } while (0)
#define CKL(call)                                                                                  \
  do { CK(call); c->launches++; } while (0)
// launch of a profiled kind: bracketed by events when that kind is selected
#define CKLK(kind, call)                                                                           \
  do {                                                                                             \
    const bool prof_ = (c->prof_mask >> (kind)) & 1u;                                              \
    if (prof_) CK(prof_mark(c, s, (kind), true));                                                  \
    CK(call);                                                                                      \
    c->launches++;                                                                                 \
    if (prof_) CK(prof_mark(c, s, (kind), false));                                                 \
  } while (0)

cudaError_t prof_mark(l2pd_ctx *c, cudaStream_t s, int kind, bool begin) {
  size_t idx = c->prof_pending_kind.size() * 2 + (begin ? 0 : 1);
  if (!begin) idx -= 2;
  while (c->prof_events.size() <= idx) {
    cudaEvent_t e;
    cudaError_t r = cudaEventCreate(&e);
    if (r != cudaSuccess) return r;
    c->prof_events.push_back(e);
  }
  if (begin) {
    cudaError_t r = cudaEventRecord(c->prof_events[idx], s);
    if (r == cudaSuccess) c->prof_pending_kind.push_back(kind);
    return r;
  }
  return cudaEventRecord(c->prof_events[idx], s);
}

void prof_collect(l2pd_ctx *c) {
  for (size_t i = 0; i < c->prof_pending_kind.size(); ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->prof_events[2 * i], c->prof_events[2 * i + 1]) == cudaSuccess) {
      c->prof_ms[c->prof_pending_kind[i]] += ms;
      c->prof_launches[c->prof_pending_kind[i]] += 1;
    }
  }
  c->prof_pending_kind.clear();
}

template <typename T>
l2pd_status dev_alloc(l2pd_ctx *c, T **p, int64_t count) {
  CK(cudaMalloc(reinterpret_cast<void **>(p), (size_t)count * sizeof(T)));
  return L2PD_OK;
}

int64_t round_up(int64_t a, int64_t b) { return (a + b - 1) / b * b; }

size_t elt(const l2pd_ctx *c) { return c->cfg.dtype == L2PD_BF16 ? 2 : 4; }

l2pd_status encode_weight_maps(l2pd_ctx *c, std::vector<TmaDesc> &dst, const std::vector<const void *> &w,
                               int64_t rows, int64_t cols, int box_rows) {
  dst.resize(w.size());
  for (size_t l = 0; l < w.size(); ++l) {
    l2pd_status s = make_tma_2d_bf16(&dst[l], w[l], rows, cols, box_rows);
    if (s != L2PD_OK) return set_err(c, s, "tensor map encode failed (rows %lld cols %lld box %d)", (long long)rows, (long long)cols, box_rows);
  }
  return L2PD_OK;
}

// One GEMM of the step, dispatched by dtype.
template <typename T>
l2pd_status run_gemm_simt(l2pd_ctx *c, cudaStream_t s, int kind, int epi, const void *A, const void *W,
                          const void *W2, void *out, const float *bias, int M, int N, int K) {
  CKLK(kind, launch_simt_gemm<T>(s, epi, (const T *)A, (const T *)W, (const T *)W2, out, bias, M, N, K));
  return L2PD_OK;
}

int64_t round_up(int64_t a, int64_t b);

GemmArgs make_gemm_args(l2pd_ctx *c, int epi, const TmaDesc *a, const TmaDesc *b, const TmaDesc *b2, const TmaDesc *cm,
                        void *out, int M, int N, int K, const GemmPlan &pl) {
  GemmArgs g{};
  if (epi == EPI_RESIDUAL && c->ksum && effective_k_splits(K, pl.k_splits) > 1) { g.part = c->ksum; g.part_rows = (int)round_up(M, 512); }
  g.epi = epi; g.a = a; g.b = b; g.b2 = b2; g.c = cm; g.M = M; g.N = N; g.K = K; g.tile_n = pl.tile_n; g.out = out;
  g.cta_group = pl.cta_group; g.k_splits = pl.k_splits; g.slabs = pl.slabs; g.k_interleave = pl.k_interleave;
  g.status = c->d_status;
  if (M <= 128 && pl.slabs == 1 && c->a_box > 0 && c->a_box < 128) {   // few rows: the map of the same buffer with the small box
    g.a = a == &c->ta_n ? &c->ta_n_s : a == &c->ta_att ? &c->ta_att_s : a == &c->ta_h ? &c->ta_h_s : a;
    if (g.a != a) g.a_box_rows = c->a_box;
  }
  if (epi == EPI_QKV_ROPE) {
    g.rope_cols = 2 * c->cfg.n_heads * c->cfg.head_dim; g.rope_dh = c->cfg.head_dim;
    g.cs_table = c->cs_table_t; g.cs_stride = c->cfg.max_seq; g.row_pos = c->d_row_pos;
  }
  return g;
}

l2pd_status run_gemm_tc(l2pd_ctx *c, cudaStream_t s, int kind, int epi, const TmaDesc *a, const TmaDesc *b,
                        const TmaDesc *b2, const TmaDesc *cm, void *out, int M, int N, int K, const GemmPlan &pl) {
  const GemmArgs g = make_gemm_args(c, epi, a, b, b2, cm, out, M, N, K, pl);
  CKLK(kind, launch_gemm_tcgen05(s, g, c->num_sms));
  return L2PD_OK;
}

template <typename T>
l2pd_status forward_and_decide(l2pd_ctx *c, cudaStream_t s, int n_slots, int T_rows, int max_q_rows, int max_kv,
                               const l2pd_step_out *out) {
  const l2pd_config &f = c->cfg;
  const int d = f.d_model, H = f.n_heads, dh = f.head_dim, hd = H * dh, F = f.d_ff, V = f.vocab, sb = f.block_len;
  const bool tc = (f.dtype == L2PD_BF16) && !c->force_simt;
  T *n = (T *)c->n, *qkv = (T *)c->qkv, *q = (T *)c->q, *att = (T *)c->att, *hbuf = (T *)c->h, *nf = (T *)c->nf;

  if (tc) {
    // the tiling follows the row count of this step; weight tensor maps are re-encoded when the
    // box (rows of the weight tile one CTA loads) changes
    // contexts that can chain the projections of a layer into one launch keep every tile at most CHAIN_TILE_N wide:
    // the chained kernel has one ring for all of them, and that width leaves it five stages
    const int max_tn = (c->chain_clusters > 0 && T_rows > 256 && T_rows <= CHAIN_MAX_ROWS && T_rows <= c->ksum_rows) ? CHAIN_TILE_N : 256;
    // steps of at most 256 rows chain with one row slab per unit (key/value-cache configurations: the rotation is a kernel
    // of its own there); their tiling is used only when chaining is asked for
    const bool small_chain = c->chain_mode != 0 && c->chain_clusters > 0 && c->ksum && T_rows <= 256 && !c->fuse_rope;
    {
      const int abox = T_rows <= 128 ? (int)round_up(T_rows, 8) : 128;
      if (abox != c->a_box) {
        if (abox < 128) {
          const int64_t mr = c->max_rows;
          if (make_tma_2d_bf16(&c->ta_n_s, c->n, mr, d, abox) || make_tma_2d_bf16(&c->ta_att_s, c->att, mr, hd, abox) ||
              make_tma_2d_bf16(&c->ta_h_s, c->h, mr, F, abox))
            return set_err(c, L2PD_ERR_CUDA, "tensor map encode failed (activation box of %d rows)", abox);
        }
        c->a_box = abox;
        c->chain_tab_rows = -1;
      }
    }
    const int max_ks = (c->ksum == nullptr || T_rows <= c->ksum_rows) ? 4 : 1;   // K slices need their partial-sum area
    if (small_chain) {
      c->pl_qkv = plan_gemm_pair_one_slab(EPI_STORE, T_rows, 3 * hd, d, c->num_sms, 1, CHAIN_TILE_N);
      c->pl_o = plan_gemm_pair_one_slab(EPI_RESIDUAL, T_rows, d, hd, c->num_sms, max_ks, CHAIN_TILE_N);
      c->pl_down = plan_gemm_pair_one_slab(EPI_RESIDUAL, T_rows, d, F, c->num_sms, max_ks, CHAIN_TILE_N);
      c->pl_gu = plan_gemm_pair_one_slab(EPI_SWIGLU, T_rows, F, d, c->num_sms, 1, CHAIN_TILE_N);
    } else {
      c->pl_qkv = plan_gemm(EPI_STORE, T_rows, 3 * hd, d, c->num_sms, 0, 4, max_tn);
      c->pl_o = plan_gemm(EPI_RESIDUAL, T_rows, d, hd, c->num_sms, 0, max_ks, max_tn);
      c->pl_down = plan_gemm(EPI_RESIDUAL, T_rows, d, F, c->num_sms, 0, max_ks, max_tn);
      c->pl_gu = plan_gemm(EPI_SWIGLU, T_rows, F, d, c->num_sms, 0, 4, max_tn);
    }
    int box = c->pl_qkv.tile_n / c->pl_qkv.cta_group;
    if (box != c->box_qkv) { l2pd_status r = encode_weight_maps(c, c->tb_qkv, c->wqkv, 3 * hd, d, box); if (r) return r; c->box_qkv = box; }
    box = c->pl_o.tile_n / c->pl_o.cta_group;
    if (box != c->box_o) { l2pd_status r = encode_weight_maps(c, c->tb_o, c->wo, d, hd, box); if (r) return r; c->box_o = box; }
    box = c->pl_down.tile_n / c->pl_down.cta_group;
    if (box != c->box_down) { l2pd_status r = encode_weight_maps(c, c->tb_down, c->w_down, d, F, box); if (r) return r; c->box_down = box; }
    box = c->pl_gu.tile_n / 2;
    if (box != c->box_gu) {
      l2pd_status r = encode_weight_maps(c, c->tb_gate, c->w_gate, F, d, box); if (r) return r;
      r = encode_weight_maps(c, c->tb_up, c->w_up, F, d, box); if (r) return r;
      c->box_gu = box;
    }
    // output maps: rows = this step's row count (the TMA unit clips the rows beyond it)
    auto out_map = [&](TmaDesc &m, int &w_have, void *ptr, bool fp32, int64_t N, int w) -> l2pd_status {
      if ((w_have == w || w_have == -w) && c->tc_rows == T_rows) return L2PD_OK;
      if (N < w) { w_have = -w; return L2PD_OK; }   // a tile wider than the row: direct stores
      l2pd_status r = make_tma_out_3d(&m, ptr, fp32, T_rows, N, w);
      if (r) return set_err(c, r, "output tensor map encode failed (N %lld tile %d)", (long long)N, w);
      w_have = w;
      return L2PD_OK;
    };
    if (c->tc_rows != T_rows) { c->tcw_qkv = c->tcw_o = c->tcw_h = c->tcw_down = 0; }
    l2pd_status r = out_map(c->tc_qkv, c->tcw_qkv, c->qkv, false, 3 * hd, c->pl_qkv.tile_n); if (r) return r;
    // K-split projections store per-slice partial sums: their map covers [slices * rows rounded up to a whole unit][d] of ksum
    const int ks_o = c->ksum ? effective_k_splits(hd, c->pl_o.k_splits) : 1, ks_d = c->ksum ? effective_k_splits(F, c->pl_down.k_splits) : 1;
    const int64_t mpad = round_up(T_rows, 512);
    auto out_map_x = [&](TmaDesc &m, int &w_have, int ks, int w) -> l2pd_status {
      if (ks <= 1) return out_map(m, w_have, c->x, true, d, w);
      if ((w_have == w || w_have == -w) && c->tc_rows == T_rows) return L2PD_OK;
      if (d < w) { w_have = -w; return L2PD_OK; }
      l2pd_status r2 = make_tma_out_3d(&m, c->ksum, true, ks * mpad, d, w);
      if (r2) return set_err(c, r2, "output tensor map encode failed (partial sums, tile %d)", w);
      w_have = w;
      return L2PD_OK;
    };
    r = out_map_x(c->tc_o, c->tcw_o, ks_o, c->pl_o.tile_n); if (r) return r;
    r = out_map(c->tc_h, c->tcw_h, c->h, false, F, c->pl_gu.tile_n / 2); if (r) return r;
    r = out_map_x(c->tc_down, c->tcw_down, ks_d, c->pl_down.tile_n); if (r) return r;
    if (c->tc_rows != T_rows && c->chain_clusters > 0 && T_rows <= CHAIN_MAX_ROWS) {
      // maps of the last, narrower column tiles (-1: a tail the staged epilogue cannot take; the step then does not chain)
      auto tail_map = [&](TmaDesc &m, int &tail, void *ptr, bool fp32, int64_t rows, int64_t N, int w, int mult = 16) {
        tail = (int)(N % w);
        if (tail && ((tail % mult) || make_tma_out_tail(&m, ptr, fp32, rows, N, tail) != L2PD_OK)) tail = -1;
      };
      tail_map(c->tct_qkv, c->tail_qkv, c->qkv, false, T_rows, 3 * hd, c->pl_qkv.tile_n);
      tail_map(c->tct_o, c->tail_o, ks_o > 1 ? (void *)c->ksum : (void *)c->x, true, ks_o > 1 ? ks_o * mpad : T_rows, d, c->pl_o.tile_n);
      tail_map(c->tct_h, c->tail_h, c->h, false, T_rows, F, c->pl_gu.tile_n / 2, 8);   // SwiGLU drains 16 columns at a time: any multiple of 8
      tail_map(c->tct_down, c->tail_down, ks_d > 1 ? (void *)c->ksum : (void *)c->x, true, ks_d > 1 ? ks_d * mpad : T_rows, d, c->pl_down.tile_n);
    }
    c->tc_rows = T_rows;
  }

  CKLK(L2PD_K_OTHER, launch_build_row_map(s, c->d_meta, n_slots, c->d_row_slot, c->d_row_pos));
  CKLK(L2PD_K_EMBED, launch_embed_rmsnorm<T>(s, c->d_tokens, c->P + c->G, c->d_meta, c->d_row_slot, (const T *)c->tok_emb,
                              c->norm1[0], f.rms_eps, c->x, n, T_rows, d));
  if (c->cap) CK(cudaMemcpyAsync(c->cap, c->x, (size_t)T_rows * d * 4, cudaMemcpyDeviceToDevice, s));

  // The chained form of the layer loop: QKV of layer 0 alone, then per layer the attention kernel and ONE launch that
  // runs O, RMSNorm, gate/up, down and (but for the last layer) the next layer's RMSNorm and QKV.
  bool chain = false;
  const int epi_qkv = c->fuse_rope ? EPI_QKV_ROPE : EPI_STORE;
  if (tc && c->chain_mode == 1 && c->chain_clusters > 0 && c->ksum && !c->cap && f.n_layers > 0 && T_rows <= c->ksum_rows &&
      T_rows <= CHAIN_MAX_ROWS && (c->fuse_rope || c->attn_tc)) {
    // SM pairs throughout: two row slabs per unit, or one slab with the two MMA issuers on alternate k-blocks
    auto chainable = [](const GemmPlan &p) { return p.cta_group == 2 && ((p.slabs == 2 && !p.k_interleave) || (p.slabs == 1 && p.k_interleave)); };
    chain = chainable(c->pl_qkv) && chainable(c->pl_o) && chainable(c->pl_gu) && chainable(c->pl_down) &&
            c->tcw_qkv > 0 && c->tcw_o > 0 && c->tcw_h > 0 && c->tcw_down > 0 &&
            c->tail_qkv >= 0 && c->tail_o >= 0 && c->tail_h >= 0 && c->tail_down >= 0;
  }
  // the projections of layer l as steps of a chained launch (with the maps of their tail tiles)
  auto chain_gemm = [&](int which, int l) {
    ChainStep st{};
    switch (which) {
      case 0: st.g = make_gemm_args(c, epi_qkv, &c->ta_n, &c->tb_qkv[l], nullptr, &c->tc_qkv, qkv, T_rows, 3 * hd, d, c->pl_qkv);
              st.g.c_tail = c->tail_qkv > 0 ? &c->tct_qkv : nullptr; st.g.tail_cols = c->tail_qkv; break;
      case 1: st.g = make_gemm_args(c, EPI_RESIDUAL, &c->ta_att, &c->tb_o[l], nullptr, &c->tc_o, c->x, T_rows, d, hd, c->pl_o);
              st.g.c_tail = c->tail_o > 0 ? &c->tct_o : nullptr; st.g.tail_cols = c->tail_o; break;
      case 2: st.g = make_gemm_args(c, EPI_SWIGLU, &c->ta_n, &c->tb_gate[l], &c->tb_up[l], &c->tc_h, hbuf, T_rows, F, d, c->pl_gu);
              st.g.c_tail = c->tail_h > 0 ? &c->tct_h : nullptr; st.g.tail_cols = c->tail_h; break;
      default: st.g = make_gemm_args(c, EPI_RESIDUAL, &c->ta_h, &c->tb_down[l], nullptr, &c->tc_down, c->x, T_rows, d, F, c->pl_down);
              st.g.c_tail = c->tail_down > 0 ? &c->tct_down : nullptr; st.g.tail_cols = c->tail_down; break;
    }
    return st;
  };
  if (chain)
    for (int i = 0; i < 4; ++i) chain = chain && chain_step_supported(chain_gemm(i, 0));
  if (chain) {
    const int ks_o = effective_k_splits(hd, c->pl_o.k_splits), ks_d = effective_k_splits(F, c->pl_down.k_splits);
    const int64_t ks_stride = (int64_t)round_up(T_rows, 512) * d;
    const int n_ctas = 2 * c->chain_clusters;
    const size_t tab_bytes = chain_table_bytes();
    if (c->chain_tab_rows != T_rows) {
      // the tables of this row count: launch 0 = QKV of layer 0; launch l + 1 = O, RMSNorm, gate/up, down of layer l and,
      // but for the last layer, RMSNorm and QKV of layer l + 1
      auto norm_step = [&](const float *gain, int n_part) {
        ChainStep st{};
        st.is_norm = 1;
        st.nm.x = c->x; st.nm.gain = gain; st.nm.eps = f.rms_eps; st.nm.n = (bf16 *)n; st.nm.rows = T_rows; st.nm.d = d;
        st.nm.part = c->ksum; st.nm.n_part = n_part > 1 ? n_part : 0; st.nm.part_stride = ks_stride;
        return st;
      };
      c->chain_tab_rows = -1;
      c->chain_info.assign(f.n_layers + 1, ChainTableInfo{});
      for (int L = 0; L <= f.n_layers; ++L) {
        ChainStep st[6] = {};
        int k = 0;
        if (L == 0) {
          st[k++] = chain_gemm(0, 0);
        } else {
          const int l = L - 1;
          st[k++] = chain_gemm(1, l);
          st[k++] = norm_step(c->norm2[l], ks_o);
          st[k++] = chain_gemm(2, l);
          st[k++] = chain_gemm(3, l);
          if (l + 1 < f.n_layers) {
            st[k++] = norm_step(c->norm1[l + 1], ks_d);
            st[k++] = chain_gemm(0, l + 1);
          }
        }
        cudaError_t e = chain_build_table(st, k, c->d_chain_bar, c->d_status, c->h_chain_tabs + (size_t)L * tab_bytes, &c->chain_info[L]);
        if (e != cudaSuccess) return set_err(c, L2PD_ERR_CUDA, "chained launch table %d: %s", L, cudaGetErrorString(e));
      }
      CK(cudaMemcpyAsync(c->d_chain_tabs, c->h_chain_tabs, (size_t)(f.n_layers + 1) * tab_bytes, cudaMemcpyHostToDevice, s));
      c->chain_tab_rows = T_rows;
    }
    auto launch_chain = [&](int L) -> l2pd_status {
      unsigned long long *tr = nullptr;
      if (c->d_chain_trace && (int64_t)(L + 1) * CHAIN_TRACE_PHASES * CHAIN_TRACE_STAMPS * n_ctas <= c->chain_trace_cap)
        tr = c->d_chain_trace + (int64_t)L * CHAIN_TRACE_PHASES * CHAIN_TRACE_STAMPS * n_ctas;
      CKLK(L2PD_K_CHAIN, launch_gemm_chain(s, c->d_chain_tabs + (size_t)L * tab_bytes, c->chain_info[L], c->chain_clusters, &c->chain_bar_base, tr));
      return L2PD_OK;
    };
    { l2pd_status r = launch_chain(0); if (r) return r; }
    for (int l = 0; l < f.n_layers; ++l) {
      if (c->fuse_rope) {
        CKLK(L2PD_K_ATTENTION, launch_attention_tc(s, c->tq_packed, c->tk_packed, c->tv_packed, c->d_meta, (bf16 *)att, hd, 0, 0, 1,
                                  n_slots, max_q_rows, H, c->d_status));
      } else {
        // key/value-cache configurations: rotation + scatter into the store, then attention over the store
        T *kc = (T *)c->kc + (f.kv_cache_mode ? (int64_t)l * c->kv_layer_stride : 0);
        T *vc = (T *)c->vc + (f.kv_cache_mode ? (int64_t)l * c->kv_layer_stride : 0);
        CKLK(L2PD_K_ROPE, launch_rope_scatter<T>(s, qkv, c->d_meta, c->d_row_slot, c->cs_table, q, kc, vc, c->kv_seq_stride, T_rows, H, dh));
        const int kv_row_base = f.kv_cache_mode ? l * f.max_batch * f.max_seq : 0;
        CKLK(L2PD_K_ATTENTION, launch_attention_tc(s, c->ta_q, c->t_kstore, c->t_vstore, c->d_meta, (bf16 *)att, hd, f.max_seq,
                                  kv_row_base, 0, n_slots, max_q_rows, H, c->d_status));
      }
      l2pd_status r = launch_chain(l + 1);
      if (r) return r;
    }
    if (ks_d > 1) CKLK(L2PD_K_OTHER, launch_add_partials(s, c->x, c->ksum, ks_d, ks_stride, T_rows, d));
    c->chain_trace_launches = f.n_layers + 1; c->chain_trace_phases = CHAIN_TRACE_PHASES; c->chain_trace_ctas = n_ctas;
  }

  for (int l = 0; l < f.n_layers && !chain; ++l) {
    T *kc = (T *)c->kc + (f.kv_cache_mode ? (int64_t)l * c->kv_layer_stride : 0);
    T *vc = (T *)c->vc + (f.kv_cache_mode ? (int64_t)l * c->kv_layer_stride : 0);
    l2pd_status r;
    if (tc) r = run_gemm_tc(c, s, L2PD_K_GEMM_QKV, c->fuse_rope ? EPI_QKV_ROPE : EPI_STORE, &c->ta_n, &c->tb_qkv[l], nullptr, c->tcw_qkv > 0 ? &c->tc_qkv : nullptr, qkv, T_rows, 3 * hd, d, c->pl_qkv);
    else r = run_gemm_simt<T>(c, s, L2PD_K_GEMM_QKV, EPI_STORE, n, c->wqkv[l], nullptr, qkv, nullptr, T_rows, 3 * hd, d);
    if (r) return r;
    if (!(tc && c->fuse_rope))
      CKLK(L2PD_K_ROPE, launch_rope_scatter<T>(s, qkv, c->d_meta, c->d_row_slot, c->cs_table, q, kc, vc, c->kv_seq_stride, T_rows, H, dh));
    if (tc && c->fuse_rope) {
      CKLK(L2PD_K_ATTENTION, launch_attention_tc(s, c->tq_packed, c->tk_packed, c->tv_packed, c->d_meta, (bf16 *)att, hd, 0, 0, 1,
                                n_slots, max_q_rows, H, c->d_status));
    } else if (tc && c->attn_tc) {
      const int kv_row_base = f.kv_cache_mode ? l * f.max_batch * f.max_seq : 0;
      CKLK(L2PD_K_ATTENTION, launch_attention_tc(s, c->ta_q, c->t_kstore, c->t_vstore, c->d_meta, (bf16 *)att, hd, f.max_seq,
                                kv_row_base, 0, n_slots, max_q_rows, H, c->d_status));
    } else if (tc) {
      CKLK(L2PD_K_ATTENTION, launch_attention_bf16(s, (const bf16 *)q, (const bf16 *)kc, (const bf16 *)vc, c->d_meta, (bf16 *)att, hd, hd,
                                c->kv_seq_stride, hd, n_slots, max_q_rows, H, dh));
    } else {
      CKLK(L2PD_K_ATTENTION, launch_simt_attention<T>(s, q, kc, vc, c->d_meta, c->d_row_slot, att, c->kv_seq_stride, T_rows, H, dh, max_kv));
    }
    if (tc) r = run_gemm_tc(c, s, L2PD_K_GEMM_O, EPI_RESIDUAL, &c->ta_att, &c->tb_o[l], nullptr, c->tcw_o > 0 ? &c->tc_o : nullptr, c->x, T_rows, d, hd, c->pl_o);
    else r = run_gemm_simt<T>(c, s, L2PD_K_GEMM_O, EPI_RESIDUAL, att, c->wo[l], nullptr, c->x, nullptr, T_rows, d, hd);
    if (r) return r;
    {
      const int ks = (tc && c->ksum) ? effective_k_splits(hd, c->pl_o.k_splits) : 1;
      CKLK(L2PD_K_RMSNORM, launch_rmsnorm<T>(s, c->x, c->norm2[l], f.rms_eps, n, T_rows, d, c->ksum, ks > 1 ? ks : 0,
                                            (int64_t)round_up(T_rows, 512) * d));
    }
    if (tc) r = run_gemm_tc(c, s, L2PD_K_GEMM_GATE_UP, EPI_SWIGLU, &c->ta_n, &c->tb_gate[l], &c->tb_up[l], c->tcw_h > 0 ? &c->tc_h : nullptr, hbuf, T_rows, F, d, c->pl_gu);
    else r = run_gemm_simt<T>(c, s, L2PD_K_GEMM_GATE_UP, EPI_SWIGLU, n, c->w_gate[l], c->w_up[l], hbuf, nullptr, T_rows, F, d);
    if (r) return r;
    if (tc) r = run_gemm_tc(c, s, L2PD_K_GEMM_DOWN, EPI_RESIDUAL, &c->ta_h, &c->tb_down[l], nullptr, c->tcw_down > 0 ? &c->tc_down : nullptr, c->x, T_rows, d, F, c->pl_down);
    else r = run_gemm_simt<T>(c, s, L2PD_K_GEMM_DOWN, EPI_RESIDUAL, hbuf, c->w_down[l], nullptr, c->x, nullptr, T_rows, d, F);
    if (r) return r;
    // the down projection's K slices: summed by the next layer's RMSNorm, or right here when x is read by something else
    int ks_pend = (tc && c->ksum) ? effective_k_splits(F, c->pl_down.k_splits) : 1;
    const int64_t ks_stride = (int64_t)round_up(T_rows, 512) * d;
    if (ks_pend > 1 && (c->cap || l + 1 == f.n_layers)) {
      CKLK(L2PD_K_OTHER, launch_add_partials(s, c->x, c->ksum, ks_pend, ks_stride, T_rows, d));
      ks_pend = 1;
    }
    if (c->cap)
      CK(cudaMemcpyAsync(c->cap + (int64_t)(l + 1) * c->cap_stride, c->x, (size_t)T_rows * d * 4, cudaMemcpyDeviceToDevice, s));
    if (l + 1 < f.n_layers)
      CKLK(L2PD_K_RMSNORM, launch_rmsnorm<T>(s, c->x, c->norm1[l + 1], f.rms_eps, n, T_rows, d, c->ksum, ks_pend > 1 ? ks_pend : 0,
                                            ks_stride));
  }

  // confidence head on the current block's rows
  const int R = n_slots * sb;
  const int rows_padded = tc ? (int)round_up(R, 128) : R;
  CKLK(L2PD_K_FINAL_NORM, launch_final_norm_gather<T>(s, c->x, c->d_meta, c->final_norm, f.rms_eps, nf, n_slots, sb, rows_padded, d));
  int n_tiles = 1;
  float *part_m, *part_s;
  int32_t *part_i;
  if (tc) {
    int tn = lm_head_tile_n(R, V, d, c->num_sms);
    if (tn != c->tn_lm) {
      l2pd_status r = make_tma_2d_bf16(&c->tb_lm, c->lm_head, V, d, tn);
      if (r) return set_err(c, r, "tensor map encode failed for the LM head");
      c->tn_lm = tn;
    }
    n_tiles = ceil_div(V, tn);
    part_m = c->part; part_s = part_m + (int64_t)n_tiles * rows_padded;
    part_i = (int32_t *)(part_s + (int64_t)n_tiles * rows_padded);
    const int nf_box = R <= 128 ? (int)round_up(R, 8) : 128;
    if (nf_box < 128 && nf_box != c->a_box_nf) {
      if (make_tma_2d_bf16(&c->ta_nf_s, c->nf, c->max_lm_rows, d, nf_box)) return set_err(c, L2PD_ERR_CUDA, "tensor map encode failed for the LM head's rows");
      c->a_box_nf = nf_box;
    }
    GemmArgs g{};
    g.epi = EPI_LMHEAD; g.a = nf_box < 128 ? &c->ta_nf_s : &c->ta_nf; g.a_box_rows = nf_box; g.b = &c->tb_lm; g.M = R; g.N = V; g.K = d; g.tile_n = tn;
    g.bias = c->lm_bias; g.part_m = part_m; g.part_s = part_s; g.part_i = part_i; g.rows_padded = rows_padded;
    g.logits = nullptr; g.status = c->d_status;
    float *tmp_logits = nullptr;
    if (out && out->d_logits) {
      // the debug logits are indexed by sequence; with every sequence active slot == sequence order only if
      // no sequence has dropped out, so write per slot into scratch and scatter below
      g.logits = c->logits_f32;
      tmp_logits = c->logits_f32;
    }
    CKLK(L2PD_K_LM_HEAD, launch_gemm_tcgen05(s, g, c->num_sms));
    (void)tmp_logits;
  } else {
    part_m = c->part; part_s = part_m + rows_padded; part_i = (int32_t *)(part_s + rows_padded);
    l2pd_status r = run_gemm_simt<T>(c, s, L2PD_K_LM_HEAD, EPI_STORE_F32, nf, c->lm_head, nullptr, c->logits_f32, c->lm_bias, R, V, d);
    if (r) return r;
    CKLK(L2PD_K_LM_HEAD, launch_row_softmax_partials(s, c->logits_f32, R, V, part_m, part_s, part_i));
  }
  if (out && out->d_logits) {
    for (int i = 0; i < n_slots; ++i) {
      const SeqMeta &m = c->h_meta[i];
      if (m.n_blk_rows > 0)
        CK(cudaMemcpyAsync(out->d_logits + (int64_t)m.seq * sb * V, c->logits_f32 + (int64_t)i * sb * V,
                           (size_t)m.n_blk_rows * V * 4, cudaMemcpyDeviceToDevice, s));
    }
  }

  DecideArgs a{};
  a.part_m = part_m; a.part_s = part_s; a.part_i = part_i; a.n_tiles = n_tiles; a.rows_padded = rows_padded;
  a.meta = c->d_meta; a.s = sb; a.P = c->P; a.G = c->G; a.n_blocks = c->G / sb;
  a.tokens = c->d_tokens; a.tok_stride = c->P + c->G; a.masked = c->d_masked; a.st = c->st;
  a.w1 = c->fw1; a.b1 = c->fb1; a.w2 = c->fw2; a.b2 = c->fb2; a.tau = f.tau;
  a.use_filter = f.use_filter; a.use_eotp = f.use_eotp; a.committed_conf_mode = f.committed_conf_mode;
  a.eot_id = f.eot_id; a.summary = c->d_summary;
  a.rule = c->rule; a.conf_threshold = c->conf_threshold; a.ref = c->d_ref;
  a.n_filter_layers = c->n_filter_layers;
  for (int k = 0; k < 4; ++k) { a.fw[k] = c->flt_w[k]; a.fb[k] = c->flt_b[k]; }
  if (c->n_filter_layers > 0) a.use_filter = 1;
  if (c->collect_c) {   // (capacity was checked before the step's first launch)
    a.collect_c = c->collect_c; a.collect_y = c->collect_y; a.collect_base = c->collect_n;
    c->collect_n += n_slots;
  }
  if (out) { a.o_conf = out->d_conf; a.o_pred = out->d_pred; a.o_p = out->d_p; a.o_unmask = out->d_unmask; }
  CKLK(L2PD_K_DECIDE, launch_decide(s, a, n_slots));
  return L2PD_OK;
}

void free_all(l2pd_ctx *c) {
  cudaFree(c->d_tokens); cudaFree(c->d_masked); cudaFree(c->d_state_ints);
  cudaFree(c->x); cudaFree(c->n); cudaFree(c->qkv); cudaFree(c->q); cudaFree(c->att); cudaFree(c->h); cudaFree(c->nf);
  cudaFree(c->kc); cudaFree(c->vc); cudaFree(c->part); cudaFree(c->logits_f32);
  for (void *w : c->wqkv_perm) cudaFree(w);
  cudaFree(c->d_row_pos); cudaFree(c->cs_table_t); cudaFree(c->ksum);
  cudaFree(c->d_chain_bar); cudaFree(c->d_chain_trace); cudaFree(c->d_chain_tabs);
  if (c->h_chain_tabs) cudaFreeHost(c->h_chain_tabs);
  cudaFree(c->d_meta); cudaFree(c->d_row_slot); cudaFree(c->d_summary); cudaFree(c->d_status); cudaFree(c->cs_table);
  if (c->h_meta) cudaFreeHost(c->h_meta);
  if (c->h_summary) cudaFreeHost(c->h_summary);
  if (c->h_status) cudaFreeHost(c->h_status);
  for (cudaEvent_t e : c->prof_events) cudaEventDestroy(e);
  if (c->ev0) cudaEventDestroy(c->ev0);
  if (c->ev1) cudaEventDestroy(c->ev1);
}

l2pd_status validate(const l2pd_config *f, const l2pd_weights *w, std::string *why) {
  auto bad = [&](const char *m) { *why = m; return L2PD_ERR_SHAPE; };
  if (f->dtype != L2PD_F32 && f->dtype != L2PD_BF16) { *why = "dtype must be L2PD_F32 or L2PD_BF16"; return L2PD_ERR_ARG; }
  if (f->n_layers < 0 || f->d_model <= 0 || f->n_heads <= 0 || f->head_dim <= 0 || f->d_ff <= 0 || f->vocab <= 1)
    return bad("non-positive model dimension");
  if (f->d_model % 8 || f->d_ff % 8 || (f->n_heads * f->head_dim) % 8) return bad("d_model, d_ff and n_heads*head_dim must be multiples of 8");
  if (f->head_dim % 2) return bad("head_dim must be even");
  if (f->dtype == L2PD_BF16 && f->head_dim != 64 && f->head_dim != 128) return bad("bf16 attention supports head_dim 64 or 128");
  if (f->dtype == L2PD_F32 && f->head_dim > 256) return bad("head_dim > 256");
  if (f->block_len < 1 || f->block_len > 64) return bad("block_len must be in [1, 64]");
  if (f->mask_id < 0 || f->mask_id >= f->vocab || f->eot_id < 0 || f->eot_id >= f->vocab || f->mask_id == f->eot_id)
    return bad("mask_id / eot_id outside the vocabulary or equal");
  if (f->max_batch < 1 || f->max_seq < 2) return bad("max_batch / max_seq too small");
  if (!(f->tau >= 0.f && f->tau <= 1.f)) { *why = "tau outside [0, 1]"; return L2PD_ERR_ARG; }
  if (f->kv_cache_mode < 0 || f->kv_cache_mode > 2) { *why = "kv_cache_mode must be 0, 1 or 2"; return L2PD_ERR_ARG; }
  if (f->committed_conf_mode != 0 && f->committed_conf_mode != 1) { *why = "committed_conf_mode must be 0 or 1"; return L2PD_ERR_ARG; }
  if (!(f->rms_eps >= 0.f) || !(f->rope_theta > 0.f)) { *why = "rms_eps / rope_theta"; return L2PD_ERR_ARG; }
  if (!w->tok_emb || !w->lm_head || !w->final_norm) { *why = "null weight pointer"; return L2PD_ERR_ARG; }
  if (f->n_layers > 0 && (!w->wqkv || !w->wo || !w->w_gate || !w->w_up || !w->w_down || !w->norm1 || !w->norm2)) {
    *why = "null per-layer weight array"; return L2PD_ERR_ARG;
  }
  for (int l = 0; l < f->n_layers; ++l)
    if (!w->wqkv[l] || !w->wo[l] || !w->w_gate[l] || !w->w_up[l] || !w->w_down[l] || !w->norm1[l] || !w->norm2[l]) {
      *why = "null per-layer weight pointer"; return L2PD_ERR_ARG;
    }
  if (f->use_filter && (!w->filt_w1 || !w->filt_b1 || !w->filt_w2 || !w->filt_b2)) { *why = "use_filter set but a filter pointer is null"; return L2PD_ERR_ARG; }
  return L2PD_OK;
}

}  // namespace

// what failed in the calling thread's last stand-alone call (l2pd_last_error(NULL))
static thread_local char g_standalone_err[160] = "";
namespace l2pd {
void set_standalone_error(const char *fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_standalone_err, sizeof(g_standalone_err), fmt, ap);
  va_end(ap);
}
}  // namespace l2pd

extern "C" {

l2pd_status l2pd_init(const l2pd_config *cfg, const l2pd_weights *w, int device, l2pd_ctx **out) {
  if (out) *out = nullptr;
  if (!cfg || !w || !out) return L2PD_ERR_ARG;
  std::string why;
  l2pd_status vs = validate(cfg, w, &why);
  if (vs != L2PD_OK) return vs;
  l2pd_ctx *c = new (std::nothrow) l2pd_ctx();
  if (!c) return L2PD_ERR_OOM;
  c->cfg = *cfg;
  c->device = device;
  const l2pd_config &f = c->cfg;
  auto fail = [&](l2pd_status s) { free_all(c); delete c; return s; };
  if (cudaSetDevice(device) != cudaSuccess) return fail(L2PD_ERR_CUDA);
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms <= 0) return fail(L2PD_ERR_CUDA);
  c->num_sms = sms;
  if (f.dtype == L2PD_BF16) {
    int major = 0;
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
    if (major != 10) return fail(L2PD_ERR_CUDA);   // the tensor-core kernels are sm_100a only
  }
  const char *fs = getenv("L2PD_FORCE_SIMT");
  c->force_simt = fs && fs[0] == '1';

  c->tok_emb = w->tok_emb; c->lm_head = w->lm_head; c->final_norm = w->final_norm; c->lm_bias = w->lm_head_bias;
  c->fw1 = w->filt_w1; c->fb1 = w->filt_b1; c->fw2 = w->filt_w2; c->fb2 = w->filt_b2;
  for (int l = 0; l < f.n_layers; ++l) {
    c->wqkv.push_back(w->wqkv[l]); c->wo.push_back(w->wo[l]); c->w_gate.push_back(w->w_gate[l]);
    c->w_up.push_back(w->w_up[l]); c->w_down.push_back(w->w_down[l]);
    c->norm1.push_back(w->norm1[l]); c->norm2.push_back(w->norm2[l]);
  }
  if (f.n_layers == 0) { c->norm1.push_back(w->final_norm); }

  const int d = f.d_model, hd = f.n_heads * f.head_dim, F = f.d_ff, V = f.vocab, sb = f.block_len;
  const size_t es = elt(c);
  c->max_rows = round_up((int64_t)f.max_batch * f.max_seq, 128);
  c->max_lm_rows = round_up((int64_t)f.max_batch * sb, 128);
  const int64_t mr = c->max_rows;
  l2pd_status r = L2PD_OK;
  auto A = [&](l2pd_status s) { if (r == L2PD_OK) r = s; };
  A(dev_alloc(c, &c->d_tokens, (int64_t)f.max_batch * f.max_seq));
  A(dev_alloc(c, &c->d_masked, (int64_t)f.max_batch * f.max_seq));
  A(dev_alloc(c, &c->d_state_ints, (int64_t)6 * f.max_batch));
  A(dev_alloc(c, &c->x, mr * d));
  A(dev_alloc(c, (uint8_t **)&c->n, mr * d * es));
  A(dev_alloc(c, (uint8_t **)&c->qkv, mr * 3 * hd * es));
  A(dev_alloc(c, (uint8_t **)&c->q, mr * hd * es));
  A(dev_alloc(c, (uint8_t **)&c->att, mr * hd * es));
  A(dev_alloc(c, (uint8_t **)&c->h, mr * F * es));
  A(dev_alloc(c, (uint8_t **)&c->nf, c->max_lm_rows * d * es));
  c->kv_seq_stride = (int64_t)f.max_seq * hd;
  c->kv_layer_stride = (int64_t)f.max_batch * c->kv_seq_stride;
  const int kv_layers = f.kv_cache_mode ? (f.n_layers > 0 ? f.n_layers : 1) : 1;
  A(dev_alloc(c, (uint8_t **)&c->kc, c->kv_layer_stride * kv_layers * es));
  A(dev_alloc(c, (uint8_t **)&c->vc, c->kv_layer_stride * kv_layers * es));
  c->part_tiles_cap = ceil_div(V, 64);
  A(dev_alloc(c, &c->part, 3 * c->part_tiles_cap * c->max_lm_rows));
  A(dev_alloc(c, &c->logits_f32, c->max_lm_rows * (int64_t)V));
  A(dev_alloc(c, &c->d_meta, (int64_t)f.max_batch));
  A(dev_alloc(c, &c->d_row_slot, mr));
  A(dev_alloc(c, &c->d_row_pos, mr));
  // L2PD_ATOMIC_KSPLIT=1: no partial-sum area; K slices add into x in completion order (not bit-reproducible)
  const char *ak = getenv("L2PD_ATOMIC_KSPLIT");
  if (f.dtype == L2PD_BF16 && !(ak && ak[0] == '1')) {
    c->ksum_rows = round_up(mr < 4096 ? mr : 4096, 512);   // a slice's area covers whole 512-row units
    A(dev_alloc(c, &c->ksum, 4 * c->ksum_rows * d));
  }
  if (f.dtype == L2PD_BF16 && c->ksum && !c->force_simt) {
    c->chain_clusters = chain_max_clusters(c->num_sms);
    if (c->chain_clusters > 0) {
      A(dev_alloc(c, &c->d_chain_bar, (int64_t)1));
      A(dev_alloc(c, &c->d_chain_tabs, (int64_t)(f.n_layers + 1) * (int64_t)chain_table_bytes()));
      if (r == L2PD_OK && cudaMallocHost((void **)&c->h_chain_tabs, (size_t)(f.n_layers + 1) * chain_table_bytes()) != cudaSuccess) r = L2PD_ERR_OOM;
    }
  }
  A(dev_alloc(c, &c->d_summary, (int64_t)f.max_batch));
  A(dev_alloc(c, &c->d_status, (int64_t)1));
  A(dev_alloc(c, &c->cs_table, (int64_t)f.max_seq * (f.head_dim / 2)));
  if (r != L2PD_OK) return fail(r);
  if (cudaMallocHost((void **)&c->h_meta, sizeof(SeqMeta) * f.max_batch) != cudaSuccess ||
      cudaMallocHost((void **)&c->h_summary, sizeof(StepSummary) * f.max_batch) != cudaSuccess ||
      cudaMallocHost((void **)&c->h_status, sizeof(int32_t)) != cudaSuccess)
    return fail(L2PD_ERR_OOM);
  if (cudaMemset(c->d_status, 0, 4) != cudaSuccess) return fail(L2PD_ERR_CUDA);
  if (c->d_chain_bar && cudaMemset(c->d_chain_bar, 0, 4) != cudaSuccess) return fail(L2PD_ERR_CUDA);
  // the activation buffers back TMA boxes that reach past the live rows: start them defined
  if (cudaMemset(c->n, 0, mr * d * es) != cudaSuccess || cudaMemset(c->att, 0, mr * hd * es) != cudaSuccess ||
      cudaMemset(c->h, 0, mr * F * es) != cudaSuccess || cudaMemset(c->nf, 0, c->max_lm_rows * d * es) != cudaSuccess ||
      cudaMemset(c->q, 0, mr * hd * es) != cudaSuccess || cudaMemset(c->qkv, 0, mr * 3 * hd * es) != cudaSuccess)
    return fail(L2PD_ERR_CUDA);
  // key tiles reach past a sequence's last key: what lies there is masked out of the scores, but
  // the value rows are multiplied by a probability of zero, so they must never hold NaN or Inf
  if (cudaMemset(c->kc, 0, c->kv_layer_stride * kv_layers * es) != cudaSuccess ||
      cudaMemset(c->vc, 0, c->kv_layer_stride * kv_layers * es) != cudaSuccess)
    return fail(L2PD_ERR_CUDA);
  c->st.cur_block = c->d_state_ints; c->st.l_eff = c->d_state_ints + f.max_batch;
  c->st.done = c->d_state_ints + 2 * f.max_batch; c->st.steps = c->d_state_ints + 3 * f.max_batch;
  c->st.eot_pos = c->d_state_ints + 4 * f.max_batch; c->st.forced = c->d_state_ints + 5 * f.max_batch;

  // rotary table in double precision on the host: angle(pos, i) = pos * theta^(-2i/dh)
  {
    const int half = f.head_dim / 2;
    std::vector<float2> tab((size_t)f.max_seq * half);
    for (int pos = 0; pos < f.max_seq; ++pos)
      for (int i = 0; i < half; ++i) {
        const double ang = (double)pos * pow((double)f.rope_theta, -2.0 * i / f.head_dim);
        tab[(size_t)pos * half + i] = make_float2((float)cos(ang), (float)sin(ang));
      }
    if (cudaMemcpy(c->cs_table, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice) != cudaSuccess)
      return fail(L2PD_ERR_CUDA);
    std::vector<float2> tab_t(tab.size());
    for (int pos = 0; pos < f.max_seq; ++pos)
      for (int i = 0; i < half; ++i) tab_t[(size_t)i * f.max_seq + pos] = tab[(size_t)pos * half + i];
    if (cudaMalloc((void **)&c->cs_table_t, tab_t.size() * sizeof(float2)) != cudaSuccess) return fail(L2PD_ERR_OOM);
    if (cudaMemcpy(c->cs_table_t, tab_t.data(), tab_t.size() * sizeof(float2), cudaMemcpyHostToDevice) != cudaSuccess)
      return fail(L2PD_ERR_CUDA);
  }
  if (f.dtype == L2PD_BF16) {
    l2pd_status s1 = make_tma_2d_bf16(&c->ta_n, c->n, mr, d, 128);
    l2pd_status s2 = make_tma_2d_bf16(&c->ta_att, c->att, mr, hd, 128);
    l2pd_status s3 = make_tma_2d_bf16(&c->ta_h, c->h, mr, F, 128);
    l2pd_status s4 = make_tma_2d_bf16(&c->ta_nf, c->nf, c->max_lm_rows, d, 128);
    if (s1 || s2 || s3 || s4) return fail(L2PD_ERR_CUDA);
    const char *aw = getenv("L2PD_ATTN_WARP");
    c->attn_tc = attention_tc_supported(f.head_dim, hd, hd, hd) && !(aw && aw[0] == '1');
    if (c->attn_tc) {
      const int64_t store_rows = (int64_t)kv_layers * f.max_batch * f.max_seq;
      if (make_tma_2d_bf16(&c->ta_q, c->q, mr, hd, 128) || make_tma_2d_bf16(&c->t_kstore, c->kc, store_rows, hd, 128) ||
          make_tma_2d_bf16(&c->t_vstore, c->vc, store_rows, hd, 128))
        return fail(L2PD_ERR_CUDA);
    }
    const char *nf = getenv("L2PD_NO_ROPE_FUSION");
    c->fuse_rope = c->attn_tc && !c->force_simt && f.kv_cache_mode == 0 && (f.head_dim & (f.head_dim - 1)) == 0 &&
                   !(nf && nf[0] == '1');
    if (c->fuse_rope) {
      bf16 *qkvb = (bf16 *)c->qkv;
      if (make_tma_2d_bf16_strided(&c->tq_packed, qkvb, mr, hd, 3 * hd, 128) ||
          make_tma_2d_bf16_strided(&c->tk_packed, qkvb + hd, mr, hd, 3 * hd, 128) ||
          make_tma_2d_bf16_strided(&c->tv_packed, qkvb + 2 * hd, mr, hd, 3 * hd, 128))
        return fail(L2PD_ERR_CUDA);
      for (int l = 0; l < f.n_layers; ++l) {
        void *w = nullptr;
        if (cudaMalloc(&w, (size_t)3 * hd * d * 2) != cudaSuccess) return fail(L2PD_ERR_OOM);
        c->wqkv_perm.push_back(w);
        if (launch_permute_qkv_rows(0, (const bf16 *)c->wqkv[l], (bf16 *)w, f.n_heads, f.head_dim, d) != cudaSuccess)
          return fail(L2PD_ERR_CUDA);
        c->wqkv[l] = w;   // the tensor maps of the QKV projection are encoded over the reordered copy
      }
      if (cudaDeviceSynchronize() != cudaSuccess) return fail(L2PD_ERR_CUDA);
    }
  }
  if (cudaEventCreate(&c->ev0) != cudaSuccess || cudaEventCreate(&c->ev1) != cudaSuccess) return fail(L2PD_ERR_CUDA);
  c->h_cur_block.assign(f.max_batch, 0); c->h_l_eff.assign(f.max_batch, 0); c->h_done.assign(f.max_batch, 1);
  c->h_steps.assign(f.max_batch, 0); c->h_cache_block.assign(f.max_batch, -1);
  *out = c;
  return L2PD_OK;
}

l2pd_status l2pd_state_reset(l2pd_ctx *c, void *stream, const int32_t *d_prompts, int32_t B, int32_t P, int32_t G) {
  if (!c || !d_prompts) return set_err(c, L2PD_ERR_ARG, "null argument");
  const l2pd_config &f = c->cfg;
  if (B < 1 || B > f.max_batch) return set_err(c, L2PD_ERR_SHAPE, "batch %d outside [1, %d]", B, f.max_batch);
  if (P < 1 || G < 1 || P + G > f.max_seq) return set_err(c, L2PD_ERR_SHAPE, "P + G = %d exceeds max_seq %d (or P, G < 1)", P + G, f.max_seq);
  if (G % f.block_len) return set_err(c, L2PD_ERR_SHAPE, "generation length %d is not a multiple of the block length %d", G, f.block_len);
  if (c->rule == L2PD_RULE_EGP && (B > c->ref_rows || G != c->ref_len))
    return set_err(c, L2PD_ERR_SHAPE, "reference answers are [%d, %d]; the reset asks for B = %d, G = %d", c->ref_rows, c->ref_len, B, G);
  cudaStream_t s = (cudaStream_t)stream;
  CK(cudaSetDevice(c->device));
  c->has_state = false;
  int32_t *d_bad = c->d_status;   // reused as the range-check flag for this call
  CK(cudaMemsetAsync(d_bad, 0, 4, s));
  CKL(launch_state_reset(s, d_prompts, B, P, G, f.vocab, f.mask_id, c->d_tokens, c->d_masked, c->st, d_bad));
  CK(cudaMemcpyAsync(c->h_status, d_bad, 4, cudaMemcpyDeviceToHost, s));
  CK(cudaMemsetAsync(d_bad, 0, 4, s));
  CK(cudaStreamSynchronize(s));
  if (*c->h_status) return set_err(c, L2PD_ERR_TOKEN_RANGE, "a prompt id is outside [0, vocab) or equals mask_id");
  c->B = B; c->P = P; c->G = G;
  for (int i = 0; i < B; ++i) { c->h_cur_block[i] = 0; c->h_l_eff[i] = P + G; c->h_done[i] = 0; c->h_steps[i] = 0; c->h_cache_block[i] = -1; }
  c->n_active = B;
  c->total_steps = 0;
  c->has_state = true;
  return L2PD_OK;
}

l2pd_status l2pd_denoise_step(l2pd_ctx *c, void *stream, const l2pd_step_out *out) {
  if (!c) return L2PD_ERR_ARG;
  if (!c->has_state || c->n_active == 0) return set_err(c, L2PD_ERR_STATE, "no unfinished sequence (reset first)");
  const l2pd_config &f = c->cfg;
  cudaStream_t s = (cudaStream_t)stream;
  CK(cudaSetDevice(c->device));
  const int sb = f.block_len;
  int n_slots = 0, T_rows = 0, max_q = 0, max_kv = 0;
  for (int i = 0; i < c->B; ++i) {
    if (c->h_done[i]) continue;
    SeqMeta &m = c->h_meta[n_slots++];
    const int b = c->h_cur_block[i], S_b = c->P + b * sb, L = c->h_l_eff[i];
    const bool cached = f.kv_cache_mode != 0 && c->h_cache_block[i] == b;
    m.seq = i; m.row0 = T_rows; m.pos0 = cached ? S_b : 0; m.n_rows = L - m.pos0; m.kv_len = L;
    m.blk_start = S_b; m.n_blk_rows = (L - S_b < sb) ? (L - S_b) : sb; m.block = b;
    // dual cache: a cached step computes the block's rows only; their K/V overwrite the store in place and the
    // positions after the block are read as the block's first step left them
    if (cached && f.kv_cache_mode == 2) m.n_rows = m.n_blk_rows;
    if (f.kv_cache_mode != 0) c->h_cache_block[i] = b;
    T_rows += m.n_rows;
    if (m.n_rows > max_q) max_q = m.n_rows;
    if (L > max_kv) max_kv = L;
  }
  c->last_rows = T_rows;
  if (c->collect_c && c->collect_n + n_slots > c->collect_cap)   // a full sink: nothing is launched, nothing appended
    return set_err(c, L2PD_ERR_SHAPE, "sample sink full (%lld of %lld)", (long long)c->collect_n, (long long)c->collect_cap);
  CK(cudaEventRecord(c->ev0, s));
  CK(cudaMemcpyAsync(c->d_meta, c->h_meta, sizeof(SeqMeta) * n_slots, cudaMemcpyHostToDevice, s));
  l2pd_status r = (f.dtype == L2PD_BF16) ? forward_and_decide<bf16>(c, s, n_slots, T_rows, max_q, max_kv, out)
                                         : forward_and_decide<float>(c, s, n_slots, T_rows, max_q, max_kv, out);
  if (r != L2PD_OK) return r;
  CK(cudaMemcpyAsync(c->h_summary, c->d_summary, sizeof(StepSummary) * c->B, cudaMemcpyDeviceToHost, s));
  CK(cudaMemcpyAsync(c->h_status, c->d_status, 4, cudaMemcpyDeviceToHost, s));
  CK(cudaEventRecord(c->ev1, s));
  CK(cudaStreamSynchronize(s));
  CK(cudaEventElapsedTime(&c->last_ms, c->ev0, c->ev1));
  prof_collect(c);
  if (*c->h_status != DEV_OK) {
    const int code = *c->h_status;
    cudaMemsetAsync(c->d_status, 0, 4, s);
    if (c->d_chain_bar) { cudaMemsetAsync(c->d_chain_bar, 0, 4, s); c->chain_bar_base = 0; }   // the meeting counter stopped short
    return set_err(c, L2PD_ERR_TIMEOUT, "a bounded device wait ran out (role %d)", code);
  }
  c->total_steps++;
  for (int k = 0; k < n_slots; ++k) {
    const int i = c->h_meta[k].seq;
    const StepSummary &sm = c->h_summary[i];
    c->h_cur_block[i] = sm.cur_block; c->h_l_eff[i] = sm.l_eff; c->h_done[i] = sm.done; c->h_steps[i]++;
    if (sm.done) c->n_active--;
    if (out) {
      if (out->h_block) out->h_block[i] = sm.block;
      if (out->h_masks_left) out->h_masks_left[i] = sm.masks_left;
      if (out->h_l_eff) out->h_l_eff[i] = sm.l_eff;
      if (out->h_done) out->h_done[i] = sm.done;
      if (out->h_forced) out->h_forced[i] = sm.forced;
    }
  }
  return L2PD_OK;
}

l2pd_status l2pd_decode(l2pd_ctx *c, void *stream, const int32_t *d_prompts, int32_t B, int32_t P, int32_t G,
                        int32_t *d_out_tokens, int32_t *h_out_len, int32_t *h_steps, int32_t *h_total_steps) {
  if (!c || !d_out_tokens) return set_err(c, L2PD_ERR_ARG, "null argument");
  l2pd_status r = l2pd_state_reset(c, stream, d_prompts, B, P, G);
  if (r != L2PD_OK) return r;
  const int64_t cap = (int64_t)B * G + 1;   // the progress fallback bounds a sequence by G steps
  int64_t it = 0;
  while (c->n_active > 0) {
    if (++it > cap) return set_err(c, L2PD_ERR_STATE, "decode did not finish within B*G steps");
    r = l2pd_denoise_step(c, stream, nullptr);
    if (r != L2PD_OK) return r;
  }
  cudaStream_t s = (cudaStream_t)stream;
  CKL(launch_gather_response(s, c->d_tokens, B, P, G, d_out_tokens));
  CK(cudaStreamSynchronize(s));
  for (int i = 0; i < B; ++i) {
    if (h_out_len) h_out_len[i] = c->h_l_eff[i] - P;
    if (h_steps) h_steps[i] = c->h_steps[i];
  }
  if (h_total_steps) *h_total_steps = c->total_steps;
  return L2PD_OK;
}

l2pd_status l2pd_set_unmask_rule(l2pd_ctx *c, void *stream, int32_t rule, float conf_threshold,
                                 const int32_t *d_reference, int32_t ref_rows, int32_t ref_len) {
  if (!c) return L2PD_ERR_ARG;
  if (rule != L2PD_RULE_FILTER && rule != L2PD_RULE_CONFIDENCE && rule != L2PD_RULE_EGP)
    return set_err(c, L2PD_ERR_ARG, "unknown rule %d", rule);
  if (rule == L2PD_RULE_CONFIDENCE && !(conf_threshold >= 0.f && conf_threshold <= 1.f))
    return set_err(c, L2PD_ERR_ARG, "confidence threshold %g outside [0, 1]", (double)conf_threshold);
  if (rule == L2PD_RULE_EGP) {
    if (!d_reference || ref_rows < 1 || ref_len < 1) return set_err(c, L2PD_ERR_ARG, "rule EGP needs reference answers");
    cudaStream_t s = (cudaStream_t)stream;
    CK(cudaSetDevice(c->device));
    CK(cudaMemsetAsync(c->d_status, 0, 4, s));
    CKL(launch_check_ids(s, d_reference, (int64_t)ref_rows * ref_len, c->cfg.vocab, c->cfg.mask_id, c->d_status));
    CK(cudaMemcpyAsync(c->h_status, c->d_status, 4, cudaMemcpyDeviceToHost, s));
    CK(cudaMemsetAsync(c->d_status, 0, 4, s));
    CK(cudaStreamSynchronize(s));
    if (*c->h_status) return set_err(c, L2PD_ERR_TOKEN_RANGE, "a reference id is outside [0, vocab) or equals mask_id");
  }
  c->has_state = false;   // the next decode starts from a reset
  c->n_active = 0;
  c->rule = rule;
  if (rule == L2PD_RULE_CONFIDENCE) c->conf_threshold = conf_threshold;
  c->d_ref = rule == L2PD_RULE_EGP ? d_reference : nullptr;
  c->ref_rows = rule == L2PD_RULE_EGP ? ref_rows : 0;
  c->ref_len = rule == L2PD_RULE_EGP ? ref_len : 0;
  return L2PD_OK;
}

l2pd_status l2pd_set_filter(l2pd_ctx *c, int32_t n_layers, const float *const *d_w, const float *const *d_b) {
  if (!c) return L2PD_ERR_ARG;
  if (n_layers < 0 || n_layers > 4) return set_err(c, L2PD_ERR_ARG, "filter depth %d outside [0, 4]", n_layers);
  for (int k = 0; k < n_layers; ++k)
    if (!d_w || !d_b || !d_w[k] || !d_b[k]) return set_err(c, L2PD_ERR_ARG, "filter layer %d: null pointer", k);
  c->n_filter_layers = n_layers;
  for (int k = 0; k < 4; ++k) { c->flt_w[k] = k < n_layers ? d_w[k] : nullptr; c->flt_b[k] = k < n_layers ? d_b[k] : nullptr; }
  return L2PD_OK;
}

l2pd_status l2pd_set_collect(l2pd_ctx *c, float *d_c, uint8_t *d_y, int64_t capacity) {
  if (!c) return L2PD_ERR_ARG;
  if ((d_c == nullptr) != (d_y == nullptr) || (d_c && capacity < 1)) return set_err(c, L2PD_ERR_ARG, "sample sink: both arrays and a capacity, or neither");
  c->collect_c = d_c; c->collect_y = d_y; c->collect_cap = d_c ? capacity : 0; c->collect_n = 0;
  return L2PD_OK;
}
int64_t l2pd_collect_count(const l2pd_ctx *c) { return c ? c->collect_n : 0; }

static l2pd_status filter_train_impl(void *stream, int32_t s, int32_t L, int64_t N, const float *d_c, const uint8_t *d_y,
                                     float *const *w, float *const *b, const l2pd_train_config *t, float *h_losses) {
  if (!d_c || !d_y || !w || !b || !t) return L2PD_ERR_ARG;
  if (L < 1 || L > 4) return L2PD_ERR_ARG;
  for (int k = 0; k < L; ++k) if (!w[k] || !b[k]) return L2PD_ERR_ARG;
  if (s < 1 || s > 64 || N < 1) return L2PD_ERR_SHAPE;
  if (t->epochs < 0 || t->batch_size < 0 || !(t->lr > 0.f) || !(t->beta1 >= 0.f && t->beta1 < 1.f) ||
      !(t->beta2 >= 0.f && t->beta2 < 1.f) || !(t->eps > 0.f) || !(t->weight_decay >= 0.f)) return L2PD_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return L2PD_ERR_CUDA;
  const int per = s * s + s, P = L * per;
  const int64_t bs = t->batch_size > 0 ? t->batch_size : N;
  const int64_t per_epoch = (N + bs - 1) / bs, updates = per_epoch * t->epochs;
  float *theta = nullptr, *gpart = nullptr, *losses = nullptr;
  auto cleanup = [&]() { cudaFree(theta); cudaFree(gpart); cudaFree(losses); };
  if (cudaMalloc(&theta, sizeof(float) * 3 * P) != cudaSuccess || cudaMalloc(&gpart, sizeof(float) * (size_t)sms * (P + 1)) != cudaSuccess ||
      cudaMalloc(&losses, sizeof(float) * (size_t)(updates > 0 ? updates : 1)) != cudaSuccess) { cleanup(); return L2PD_ERR_OOM; }
  float *m = theta + P, *v = theta + 2 * P;
  const size_t ss = sizeof(float) * s * s, sv = sizeof(float) * s;
  bool ok = cudaMemsetAsync(m, 0, sizeof(float) * 2 * P, st) == cudaSuccess;
  for (int k = 0; ok && k < L; ++k)
    ok = cudaMemcpyAsync(theta + k * per, w[k], ss, cudaMemcpyDeviceToDevice, st) == cudaSuccess &&
         cudaMemcpyAsync(theta + k * per + s * s, b[k], sv, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  FilterTrainHyper h{t->lr, t->beta1, t->beta2, t->eps, t->weight_decay};
  double p1 = 1.0, p2 = 1.0;   // beta^t, carried in double
  int64_t u = 0;
  for (int e = 0; ok && e < t->epochs; ++e)
    for (int64_t lo = 0; ok && lo < N; lo += bs, ++u) {
      p1 *= t->beta1; p2 *= t->beta2;
      ok = launch_filter_update(st, d_c, d_y, lo, (N - lo < bs ? N - lo : bs), s, L, theta, m, v, gpart, sms, h, 1.0 - p1, 1.0 - p2,
                                losses + u) == cudaSuccess;
    }
  for (int k = 0; ok && k < L; ++k)
    ok = cudaMemcpyAsync(w[k], theta + k * per, ss, cudaMemcpyDeviceToDevice, st) == cudaSuccess &&
         cudaMemcpyAsync(b[k], theta + k * per + s * s, sv, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (ok && h_losses && updates > 0) ok = cudaMemcpyAsync(h_losses, losses, sizeof(float) * updates, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok = (cudaStreamSynchronize(st) == cudaSuccess) && ok;
  cleanup();
  return ok ? L2PD_OK : L2PD_ERR_CUDA;
}

l2pd_status l2pd_filter_train(void *stream, int32_t s, int64_t N, const float *d_c, const uint8_t *d_y, float *d_w1,
                              float *d_b1, float *d_w2, float *d_b2, const l2pd_train_config *t, float *h_losses) {
  float *w[2] = {d_w1, d_w2}, *b[2] = {d_b1, d_b2};
  return filter_train_impl(stream, s, 2, N, d_c, d_y, w, b, t, h_losses);
}

l2pd_status l2pd_filter_train_layers(void *stream, int32_t s, int32_t n_layers, int64_t N, const float *d_c, const uint8_t *d_y,
                                     float *const *d_w, float *const *d_b, const l2pd_train_config *t, float *h_losses) {
  return filter_train_impl(stream, s, n_layers, N, d_c, d_y, d_w, d_b, t, h_losses);
}

int32_t l2pd_num_active(const l2pd_ctx *c) { return c ? c->n_active : 0; }
const int32_t *l2pd_state_tokens(const l2pd_ctx *c) { return c ? c->d_tokens : nullptr; }
const uint8_t *l2pd_state_masked(const l2pd_ctx *c) { return c ? c->d_masked : nullptr; }

l2pd_status l2pd_set_capture(l2pd_ctx *c, float *d_resid, int64_t slot_stride_elems) {
  if (!c) return L2PD_ERR_ARG;
  if (d_resid && slot_stride_elems < (int64_t)c->cfg.d_model) return set_err(c, L2PD_ERR_SHAPE, "capture slot stride too small");
  c->cap = d_resid;
  c->cap_stride = slot_stride_elems;
  return L2PD_OK;
}
int32_t l2pd_last_step_rows(const l2pd_ctx *c) { return c ? c->last_rows : 0; }
int64_t l2pd_launch_count(const l2pd_ctx *c) { return c ? c->launches : 0; }
float l2pd_last_step_ms(const l2pd_ctx *c) { return c ? c->last_ms : -1.f; }
l2pd_status l2pd_profile_enable(l2pd_ctx *c, uint32_t kind_mask) {
  if (!c) return L2PD_ERR_ARG;
  c->prof_mask = kind_mask & ((1u << L2PD_K_COUNT) - 1u);
  c->prof_pending_kind.clear();
  for (int k = 0; k < L2PD_K_COUNT; ++k) { c->prof_ms[k] = 0.0; c->prof_launches[k] = 0; }
  return L2PD_OK;
}
l2pd_status l2pd_profile_read(const l2pd_ctx *c, int32_t kind, double *ms_total, int64_t *launches) {
  if (!c || kind < 0 || kind >= L2PD_K_COUNT) return L2PD_ERR_ARG;
  if (ms_total) *ms_total = c->prof_ms[kind];
  if (launches) *launches = c->prof_launches[kind];
  return L2PD_OK;
}
const char *l2pd_last_error(const l2pd_ctx *c);

l2pd_status l2pd_debug_set_device_status(l2pd_ctx *c, void *stream, int32_t code) {
  if (!c) return L2PD_ERR_ARG;
  CK(cudaSetDevice(c->device));
  CK(cudaMemcpyAsync(c->d_status, &code, 4, cudaMemcpyHostToDevice, (cudaStream_t)stream));
  CK(cudaStreamSynchronize((cudaStream_t)stream));
  return L2PD_OK;
}

l2pd_status l2pd_set_chain(l2pd_ctx *c, int32_t mode) {
  if (!c) return L2PD_ERR_ARG;
  if (mode < 0 || mode > 2) return set_err(c, L2PD_ERR_ARG, "chain mode %d outside [0, 2]", mode);
  c->chain_mode = mode;
  c->tc_rows = -1;          // the tiling may change with the mode: output maps and launch tables are rebuilt
  c->chain_tab_rows = -1;
  return L2PD_OK;
}

l2pd_status l2pd_chain_trace_enable(l2pd_ctx *c, int32_t enable) {
  if (!c) return L2PD_ERR_ARG;
  CK(cudaSetDevice(c->device));
  if (!enable) {
    CK(cudaDeviceSynchronize());
    cudaFree(c->d_chain_trace);
    c->d_chain_trace = nullptr; c->chain_trace_cap = 0; c->chain_trace_launches = 0;
    return L2PD_OK;
  }
  if (c->chain_clusters <= 0) return set_err(c, L2PD_ERR_STATE, "this context does not run chained launches");
  if (!c->d_chain_trace) {
    const int64_t cap = (int64_t)(c->cfg.n_layers + 1) * CHAIN_TRACE_PHASES * CHAIN_TRACE_STAMPS * (2 * c->chain_clusters);
    CK(cudaMalloc((void **)&c->d_chain_trace, (size_t)cap * 8));
    CK(cudaMemset(c->d_chain_trace, 0, (size_t)cap * 8));
    c->chain_trace_cap = cap;
  }
  c->chain_trace_launches = 0;
  return L2PD_OK;
}

int64_t l2pd_chain_trace_read(l2pd_ctx *c, uint64_t *h_out, int64_t capacity, int32_t *launches, int32_t *phases, int32_t *ctas) {
  if (!c || !c->d_chain_trace) return 0;
  if (launches) *launches = c->chain_trace_launches;
  if (phases) *phases = c->chain_trace_phases;
  if (ctas) *ctas = c->chain_trace_ctas;
  const int64_t n = (int64_t)c->chain_trace_launches * c->chain_trace_phases * CHAIN_TRACE_STAMPS * c->chain_trace_ctas;
  if (!h_out || capacity < n || n == 0) return n;
  if (cudaSetDevice(c->device) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(h_out, c->d_chain_trace, (size_t)n * 8, cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
  return n;
}

void l2pd_destroy(l2pd_ctx *c) {
  if (!c) return;
  cudaSetDevice(c->device);
  cudaDeviceSynchronize();
  free_all(c);
  delete c;
}

// ---- stand-alone kernels --------------------------------------------------------------------------------

static l2pd_status standalone_cuda_error(const char *where, cudaError_t e) {
  snprintf(g_standalone_err, sizeof(g_standalone_err), "%s: %s", where, cudaGetErrorString(e));
  return L2PD_ERR_CUDA;
}

static int32_t *standalone_status() {
  static int32_t *p[64] = {};
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!p[dev]) {
    if (cudaMalloc((void **)&p[dev], 4) != cudaSuccess) return nullptr;
    cudaMemset(p[dev], 0, 4);
  }
  return p[dev];
}

static int device_sms() {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  return sms;
}

static l2pd_status finish_standalone(cudaStream_t s, int32_t *status, int check) {
  if (!check) return L2PD_OK;
  int32_t h = 0;
  cudaError_t e = cudaMemcpyAsync(&h, status, 4, cudaMemcpyDeviceToHost, s);
  if (e != cudaSuccess) return standalone_cuda_error("status read-back", e);
  e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return standalone_cuda_error("stream synchronisation", e);
  if (h != DEV_OK) { cudaMemsetAsync(status, 0, 4, s); return L2PD_ERR_TIMEOUT; }
  return L2PD_OK;
}

static l2pd_status gemm_common(void *stream, int epi, const void *A, const void *W, const void *W2, void *out,
                               int M, int N, int K, int tile_n, int check) {
  if (!A || !W || !out || (epi == EPI_SWIGLU && !W2)) return L2PD_ERR_ARG;
  if (M < 1 || N < 8 || K < 8 || (N % 8) || (K % 8)) return L2PD_ERR_SHAPE;
  if (tile_n < 0) return L2PD_ERR_SHAPE;
  const int sms = device_sms();
  // tile_n = width + 1000 * cta_group + 10000 * k_splits + 100000 * slabs + 1000000 * k_interleave (1 = on, 2 = off);
  // any part 0 = chosen automatically
  const int want_kil = tile_n / 1000000;
  tile_n %= 1000000;
  const int want_sl = tile_n / 100000, want_ks = (tile_n % 100000) / 10000, want_cg = (tile_n % 10000) / 1000,
            want_tn = tile_n % 1000;
  const int unit = 16;
  if (want_tn && (want_tn < 32 || want_tn > 256 || (want_tn % unit))) return L2PD_ERR_SHAPE;
  if (want_cg > 2 || want_ks > 8 || (want_ks > 1 && epi != EPI_RESIDUAL) || want_sl > 2) return L2PD_ERR_SHAPE;
  GemmPlan pl = plan_gemm(epi, M, N, K, sms, want_tn);
  if (want_tn) pl.tile_n = want_tn;
  if (want_cg) pl.cta_group = want_cg;
  if (want_ks) pl.k_splits = want_ks;
  if (want_sl) pl.slabs = want_sl;
  if (want_kil == 1) pl.k_interleave = 1;
  if (want_kil == 2 || pl.slabs != 1) pl.k_interleave = 0;
  if (pl.slabs == 2 && pl.cta_group != 2) return L2PD_ERR_SHAPE;
  if (pl.k_splits > ceil_div(K, 64)) pl.k_splits = ceil_div(K, 64);
  int32_t *status = standalone_status();
  if (!status) return L2PD_ERR_CUDA;
  const int box = epi == EPI_SWIGLU ? pl.tile_n / 2 : pl.tile_n / pl.cta_group;
  TmaDesc ta, tb, tb2;
  const int a_box = (M <= 128 && pl.slabs == 1) ? (int)round_up(M, 8) : 128;   // few rows: load only those
  l2pd_status r = make_tma_2d_bf16(&ta, A, M, K, a_box);
  if (r) return r;
  r = make_tma_2d_bf16(&tb, W, N, K, box);
  if (r) return r;
  if (epi == EPI_SWIGLU) { r = make_tma_2d_bf16(&tb2, W2, N, K, box); if (r) return r; }
  // L2PD_DIRECT_STORES=1: epilogue with per-thread stores instead of the staged TMA stores (for comparison)
  static const bool direct = [] { const char *e = getenv("L2PD_DIRECT_STORES"); return e && e[0] == '1'; }();
  TmaDesc tcm;
  const int out_w = epi == EPI_SWIGLU ? pl.tile_n / 2 : pl.tile_n;
  const bool staged = !direct && N >= out_w && make_tma_out_3d(&tcm, out, epi == EPI_RESIDUAL, M, N, out_w) == L2PD_OK;
  GemmArgs g{};
  g.c = staged ? &tcm : nullptr;
  g.epi = epi; g.a = &ta; g.b = &tb; g.b2 = epi == EPI_SWIGLU ? &tb2 : nullptr;
  g.M = M; g.N = N; g.K = K; g.tile_n = pl.tile_n; g.cta_group = pl.cta_group; g.k_splits = pl.k_splits;
  g.slabs = pl.slabs; g.k_interleave = pl.k_interleave; g.a_box_rows = a_box;
  g.out = out; g.status = status;
  { cudaError_t e = launch_gemm_tcgen05((cudaStream_t)stream, g, sms); if (e != cudaSuccess) return standalone_cuda_error("GEMM launch", e); }
  return finish_standalone((cudaStream_t)stream, status, check);
}

const char *l2pd_last_error(const l2pd_ctx *c) { return c ? c->err.c_str() : g_standalone_err; }

l2pd_status l2pd_gemm_bf16(void *stream, const void *A, const void *W, void *C, int32_t M, int32_t N, int32_t K,
                           int32_t tile_n, int32_t check) {
  return gemm_common(stream, EPI_STORE, A, W, nullptr, C, M, N, K, tile_n, check);
}
l2pd_status l2pd_gemm_bf16_residual(void *stream, const void *A, const void *W, float *X, int32_t M, int32_t N,
                                    int32_t K, int32_t tile_n, int32_t check) {
  return gemm_common(stream, EPI_RESIDUAL, A, W, nullptr, X, M, N, K, tile_n, check);
}
l2pd_status l2pd_gemm_bf16_swiglu(void *stream, const void *A, const void *Wg, const void *Wu, void *H, int32_t M,
                                  int32_t F, int32_t K, int32_t tile_n, int32_t check) {
  return gemm_common(stream, EPI_SWIGLU, A, Wg, Wu, H, M, F, K, tile_n, check);
}

int64_t l2pd_lm_head_scratch_elems(int32_t R, int32_t V) {
  if (R < 1 || V < 1) return 0;
  return 3 * (int64_t)ceil_div(V, 64) * round_up(R, 128);
}

l2pd_status l2pd_lm_head_bf16(void *stream, const void *A, const void *W, const float *bias, int32_t R, int32_t V,
                              int32_t K, float *d_scratch, int32_t *d_pred, float *d_conf, float *d_logits,
                              int32_t check) {
  if (!A || !W || !d_scratch || !d_pred || !d_conf) return L2PD_ERR_ARG;
  if (R < 1 || V < 2 || K < 8 || (K % 8)) return L2PD_ERR_SHAPE;
  const int sms = device_sms();
  const int tile_n = lm_head_tile_n(R, V, K, sms);
  int32_t *status = standalone_status();
  if (!status) return L2PD_ERR_CUDA;
  TmaDesc ta, tb;
  const int a_box = R <= 128 ? (int)round_up(R, 8) : 128;
  l2pd_status r = make_tma_2d_bf16(&ta, A, R, K, a_box);
  if (r) return r;
  r = make_tma_2d_bf16(&tb, W, V, K, tile_n);
  if (r) return r;
  const int rows_padded = (int)round_up(R, 128);
  const int n_tiles = ceil_div(V, tile_n);
  GemmArgs g{};
  g.epi = EPI_LMHEAD; g.a = &ta; g.b = &tb; g.M = R; g.N = V; g.K = K; g.tile_n = tile_n;
  g.bias = bias; g.part_m = d_scratch; g.part_s = d_scratch + (int64_t)n_tiles * rows_padded;
  g.part_i = (int32_t *)(g.part_s + (int64_t)n_tiles * rows_padded); g.rows_padded = rows_padded;
  g.logits = d_logits; g.status = status; g.a_box_rows = a_box;
  cudaStream_t s = (cudaStream_t)stream;
  if (launch_gemm_tcgen05(s, g, sms) != cudaSuccess) return L2PD_ERR_CUDA;
  if (launch_merge_partials(s, g.part_m, g.part_s, g.part_i, n_tiles, rows_padded, R, d_pred, d_conf) != cudaSuccess)
    return L2PD_ERR_CUDA;
  return finish_standalone(s, status, check);
}

l2pd_status l2pd_attention_bf16(void *stream, const void *q, const void *k, const void *v, void *out, int32_t Tq,
                                int32_t Tk, int32_t H, int32_t dh, int64_t q_stride, int64_t kv_stride,
                                int64_t out_stride, int32_t impl, int32_t check) {
  if (!q || !k || !v || !out) return L2PD_ERR_ARG;
  if (Tq < 1 || Tk < 1 || H < 1 || (dh != 64 && dh != 128) || (q_stride % 8) || (kv_stride % 8) || (out_stride % 2))
    return L2PD_ERR_SHAPE;
  if (impl != 0 && impl != 1) return L2PD_ERR_ARG;
  if (q_stride < (int64_t)H * dh || kv_stride < (int64_t)H * dh || out_stride < (int64_t)H * dh) return L2PD_ERR_SHAPE;
  if (impl == 0 && attention_tc_supported(dh, q_stride, kv_stride, out_stride)) {
    int32_t *status = standalone_status();
    if (!status) return L2PD_ERR_CUDA;
    TmaDesc tq, tk, tv;
    l2pd_status r = make_tma_2d_bf16_strided(&tq, q, Tq, (int64_t)H * dh, q_stride, 128);
    if (r) return r;
    r = make_tma_2d_bf16_strided(&tk, k, Tk, (int64_t)H * dh, kv_stride, 128);
    if (r) return r;
    r = make_tma_2d_bf16_strided(&tv, v, Tk, (int64_t)H * dh, kv_stride, 128);
    if (r) return r;
    if (launch_attention_tc((cudaStream_t)stream, tq, tk, tv, nullptr, (bf16 *)out, out_stride, 0, 0, 0, Tk, Tq, H, status) !=
        cudaSuccess)
      return L2PD_ERR_CUDA;
    return finish_standalone((cudaStream_t)stream, status, check);
  }
  cudaError_t e = launch_attention_bf16((cudaStream_t)stream, (const bf16 *)q, (const bf16 *)k, (const bf16 *)v,
                                        nullptr, (bf16 *)out, q_stride, kv_stride, 0, out_stride, Tk, Tq, H, dh);
  if (e != cudaSuccess) return L2PD_ERR_CUDA;
  if (check && cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return L2PD_ERR_CUDA;
  return L2PD_OK;
}

}  // extern "C"
