// LM head + confidence head for callers that must not allocate: the per-tile reduction records
// live in a fixed device array that is part of the library image instead of caller scratch.
#include <mutex>

#include "common.cuh"

namespace l2pd {
namespace {

constexpr int STATIC_MAX_ROWS = 128;      // R <= 128 (one row tile)
constexpr int STATIC_MAX_TILES = 2048;    // vocabulary tiles: V <= 64 * 2048 = 131072
constexpr int64_t STATIC_SCRATCH_ELEMS = 3ll * STATIC_MAX_TILES * STATIC_MAX_ROWS;   // 3 MiB of fp32/int32

// Resident on every GPU that loads the library, from load until the process exits.
static __device__ __align__(256) float g_lm_scratch[STATIC_SCRATCH_ELEMS];
static __device__ __align__(256) int32_t g_lm_status[1];   // one word per device image

// In host code the names above are host-side handles, not device addresses: the addresses the
// kernels get come from cudaGetSymbolAddress, looked up once per device with that device current.
struct DevicePtrs { float *scratch = nullptr; int32_t *status = nullptr; bool ready = false; };
DevicePtrs g_dev[64];
std::mutex g_mu;

l2pd_status device_ptrs(int dev, DevicePtrs *out) {
  std::lock_guard<std::mutex> lock(g_mu);
  DevicePtrs &d = g_dev[dev];
  if (!d.ready) {
    void *ps = nullptr, *pt = nullptr;
    if (cudaGetSymbolAddress(&ps, g_lm_scratch) != cudaSuccess) return L2PD_ERR_CUDA;
    if (cudaGetSymbolAddress(&pt, g_lm_status) != cudaSuccess) return L2PD_ERR_CUDA;
    d.scratch = static_cast<float *>(ps);
    d.status = static_cast<int32_t *>(pt);
    d.ready = true;
  }
  *out = d;
  return L2PD_OK;
}

}  // namespace
}  // namespace l2pd

using namespace l2pd;

extern "C" l2pd_status l2pd_lm_head_bf16_static(void *stream, const void *A, const void *W, const float *bias,
                                                int32_t R, int32_t V, int32_t K, int32_t *d_pred, float *d_conf,
                                                int32_t check) {
  auto bad = [](l2pd_status st, const char *what) { set_standalone_error("l2pd_lm_head_bf16_static: %s", what); return st; };
  if (!A || !W || !d_pred || !d_conf) return bad(L2PD_ERR_ARG, "null pointer");
  if (R < 1 || V < 2 || K < 8 || (K % 8)) return bad(L2PD_ERR_SHAPE, "R >= 1, V >= 2, K a positive multiple of 8");
  if (R > STATIC_MAX_ROWS || V > 64 * STATIC_MAX_TILES) return bad(L2PD_ERR_SHAPE, "beyond the built-in scratch (R <= 128, V <= 131072)");
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return bad(L2PD_ERR_CUDA, "no current device");
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return bad(L2PD_ERR_CUDA, "device attribute query failed");
  DevicePtrs ptr;
  l2pd_status r = device_ptrs(dev, &ptr);
  if (r != L2PD_OK) return bad(r, "cudaGetSymbolAddress failed for the built-in scratch");
  const int tile_n = lm_head_tile_n(R, V, K, sms);
  const int n_tiles = ceil_div(V, tile_n);
  const int rows_padded = STATIC_MAX_ROWS;
  if (tile_n < 64 || n_tiles > STATIC_MAX_TILES) return bad(L2PD_ERR_SHAPE, "tile records exceed the built-in scratch");
  TmaDesc ta, tb;
  const int a_box = (R + 7) / 8 * 8;   // R <= 128: load only the rows there are
  r = make_tma_2d_bf16(&ta, A, R, K, a_box);
  if (r) return bad(r, "tensor map of A (16-byte aligned pointer, K a multiple of 8)");
  r = make_tma_2d_bf16(&tb, W, V, K, tile_n);
  if (r) return bad(r, "tensor map of W (16-byte aligned pointer, K a multiple of 8)");
  cudaStream_t s = (cudaStream_t)stream;
  // the status word must start at zero; every record the merge reads is rewritten by this call
  if (cudaMemsetAsync(ptr.status, 0, sizeof(int32_t), s) != cudaSuccess) return bad(L2PD_ERR_CUDA, "clearing the status word failed");
  GemmArgs g{};
  g.epi = EPI_LMHEAD; g.a = &ta; g.b = &tb; g.M = R; g.N = V; g.K = K; g.tile_n = tile_n;
  g.bias = bias; g.part_m = ptr.scratch; g.part_s = ptr.scratch + (int64_t)n_tiles * rows_padded;
  g.part_i = reinterpret_cast<int32_t *>(g.part_s + (int64_t)n_tiles * rows_padded);
  g.rows_padded = rows_padded; g.logits = nullptr; g.status = ptr.status; g.a_box_rows = a_box;
  if (launch_gemm_tcgen05(s, g, sms) != cudaSuccess) return bad(L2PD_ERR_CUDA, "GEMM launch failed");
  if (launch_merge_partials(s, g.part_m, g.part_s, g.part_i, n_tiles, rows_padded, R, d_pred, d_conf) != cudaSuccess)
    return bad(L2PD_ERR_CUDA, "merge launch failed");
  if (!check) return L2PD_OK;
  int32_t h = 0;
  if (cudaMemcpyAsync(&h, ptr.status, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return bad(L2PD_ERR_CUDA, "status read-back failed");
  if (cudaStreamSynchronize(s) != cudaSuccess) return bad(L2PD_ERR_CUDA, "stream synchronisation failed");
  return h == DEV_OK ? L2PD_OK : bad(L2PD_ERR_TIMEOUT, "a bounded device wait ran out");
}
