// Host side of the C ABI declared in include/laser.h: validation, workspace carve-up,
// kernel selection by E, launches.  No allocation, no synchronisation (except the host-
// buffer entry point), no state between calls.
#include "../../include/laser.h"
#include "../../include/laser_test_hooks.h"

#define LASER_DEFINE_K3_KERNEL
#include "k12_launch.cuh"
#include "k3_dispatch.cuh"
#include "k4_metrics.cuh"
#include "k5_score_stats.cuh"

using namespace laser;

namespace {

// settings of include/laser_test_hooks.h (tests only; process-wide)
int g_test_router = LASER_TEST_ROUTER_AUTO;
int g_test_withhold_tile = -1;
long long g_test_wait_cycles = 0;

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int validate_params(const laser_params* p) {
  if (!p) return LASER_ERR_INVALID_ARG;
  if (p->T < 0 || p->d <= 0 || p->E < 1 || p->E > LASER_MAX_EXPERTS) return LASER_ERR_INVALID_ARG;
  if (p->k < 1 || p->k > p->c || p->c > p->E) return LASER_ERR_INVALID_ARG;
  if (p->d % 8 != 0) return LASER_ERR_INVALID_ARG;
  if (!(p->eps_high >= 0.0f) || !(p->t_fix >= 0.0f) || !(p->t_fix <= 1.0f))
    return LASER_ERR_INVALID_ARG;
  if (p->trim_mode != 0 && p->trim_mode != 1) return LASER_ERR_INVALID_ARG;
  if (p->update_granularity < 0) return LASER_ERR_INVALID_ARG;
  if (p->update_granularity != 1 && p->update_granularity % 32 != 0) return LASER_ERR_UNSUPPORTED;
  if (p->n_bins < 1) return LASER_ERR_INVALID_ARG;
  if (p->ld_hidden < p->d || p->ld_w < p->d) return LASER_ERR_INVALID_ARG;
  if (p->ld_hidden % 8 != 0 || p->ld_w % 8 != 0) return LASER_ERR_MISALIGNED;
  if ((long long)p->T * p->k > 0x7fffffffLL) return LASER_ERR_INVALID_ARG;
  return LASER_OK;
}

// ---- tensor-memory router (E > 32): TMA tensor maps and launch --------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) !=
            cudaSuccess || q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// 2-D bf16 view [rows, d] with row pitch ld elements; boxes of box_rows x 64 elements stored
// with the 128-byte swizzle; out-of-range elements read as zero.
bool make_map(CUtensorMap* m, const void* base, long long rows, int d, long long ld, int box_rows,
              CUtensorMapL2promotion promotion) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn || rows <= 0 || rows > 0xffffffffLL) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kTcSliceK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            promotion, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// SMs of the current device (looked up once per device).
int sm_count() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

// Returns false if the tensor maps cannot be built for this call (the caller then uses the
// warp-level router, which has no such requirement).
bool launch_k12_tensor_memory(const RouteArgs& a, int n_layers, cudaStream_t s, cudaError_t* err) {
  // hidden and W_g of the layers of this launch as one [layers*T, d] / [layers*E, d] matrix
  if (a.hidden_ls != (long long)a.T * a.ld_h || a.wg_ls != (long long)a.E * a.ld_w) return false;
  const int N = a.E <= 64 ? 64 : (a.E <= 128 ? 128 : 256);
  CUtensorMap mh, mw;
  const long long total_layers = (long long)a.layer0 + n_layers;
  // the kernels address rows of these views with signed 32-bit TMA coordinates
  if (total_layers * a.T + kTcTileM > 0x7fffffffLL || total_layers * a.E > 0x7fffffffLL)
    return false;
  // hidden states are fetched from memory 256 bytes at a time (two neighbouring 128-byte rows of
  // consecutive slices): measured 7.0 instead of 5.9 TB/s for this box shape on a plain stream
  if (!make_map(&mh, a.hidden, total_layers * a.T, a.d, a.ld_h, kTcTileM,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
    return false;
  if (!make_map(&mw, a.wg, total_layers * a.E, a.d, a.ld_w, N, CU_TENSOR_MAP_L2_PROMOTION_L2_128B))
    return false;
  // E <= 64: persistent router blocks, two per SM next to the selection blocks (the one-tile-
  // per-block form stays reachable for the tests and for comparison; wider shapes have no room
  // for two such blocks per SM)
  if (N == 64 && g_test_router != LASER_TEST_ROUTER_TILE_ONESHOT) {
    *err = launch_tcp_n64(a, n_layers, 2 * sm_count() - n_layers, mh, mw, s);
    return true;
  }
  // 128 < E <= 256 with lists of at most 16: one persistent block per SM (four 48 KB stages, two
  // accumulators fill the tensor memory); the selection blocks take an SM each
  if (N == 256 && a.c <= 16 && !a.trim_random && g_test_router != LASER_TEST_ROUTER_TILE_ONESHOT) {
    int blocks = sm_count() - n_layers;
    if (blocks < sm_count() / 2) blocks = sm_count() / 2;
    *err = launch_tcp_n256(a, n_layers, blocks, mh, mw, s);
    return true;
  }
  if (N == 64) *err = launch_tc_n64(a, n_layers, mh, mw, s);
  else if (N == 128) *err = launch_tc_n128(a, n_layers, mh, mw, s);
  else *err = launch_tc_n256(a, n_layers, mh, mw, s);
  return true;
}

cudaError_t launch_k12_splitk_for_E(const RouteArgs& a, int n_layers, cudaStream_t s) {
  const int E = a.E;
  if (E <= 8) return launch_splitk_e8(a, n_layers, s);
  if (E <= 16) return launch_splitk_e16(a, n_layers, s);
  if (E <= 32) return launch_splitk_e32(a, n_layers, s);
  if (E <= 64) return launch_splitk_e64(a, n_layers, s);
  if (E <= 128) return launch_splitk_e128(a, n_layers, s);
  return launch_splitk_e256(a, n_layers, s);
}

// few tokens: 128-token tiles would leave most SMs idle, so route 16 tokens per block
// (laser_test_set_router overrides the choice for the tests)
bool use_splitk(const RouteArgs& a, int n_layers) {
  bool few = (long long)n_layers * ((a.T + 127) / 128) * 4 <= 148;
  if (g_test_router == LASER_TEST_ROUTER_TILE || g_test_router == LASER_TEST_ROUTER_TILE_ONESHOT)
    few = false;
  else if (g_test_router == LASER_TEST_ROUTER_SPLITK) few = true;
  return few;
}

// Calls of at most 7 router tiles per layer (112 tokens) whose dispatch runs inside the selection
// block are launched as one thread-block cluster per layer: no ready flags, so no memset.
int cluster_tiles_for(const RouteArgs& a, int n_layers) {
  const int tiles = (a.T + 15) / 16;
  if (!use_splitk(a, n_layers) || tiles > 7 || !a.fuse_dispatch || g_test_withhold_tile >= 0)
    return 0;
  return tiles;
}

cudaError_t launch_k12_for_E(const RouteArgs& a, int n_layers, cudaStream_t s) {
  const int E = a.E;
  if (use_splitk(a, n_layers)) return launch_k12_splitk_for_E(a, n_layers, s);
  if (E > 32) {
    cudaError_t err = cudaSuccess;
    if (launch_k12_tensor_memory(a, n_layers, s, &err)) return err;
  }
  if (E <= 8) return launch_warp_e8(a, n_layers, s);
  if (E <= 16) return launch_warp_e16(a, n_layers, s);
  if (E <= 32) return launch_warp_e32(a, n_layers, s);
  if (E <= 64) return launch_warp_e64(a, n_layers, s);
  if (E <= 128) return launch_warp_e128(a, n_layers, s);
  return launch_warp_e256(a, n_layers, s);
}

// Enqueues all stages for layers [layer0, layer0 + n) of a batched call.
int enqueue_group(RouteArgs& a, int layer0, int n, const laser_params* p, const float* eps,
                  const float* tfix, cudaStream_t s, void* const* ev) {
  auto mark = [&](int i) {
    return !ev || !ev[i] || cudaEventRecord(static_cast<cudaEvent_t>(ev[i]), s) == cudaSuccess;
  };
  a.layer0 = layer0;
  for (int l = 0; l < n; ++l) {
    a.eps_high[l] = eps ? eps[layer0 + l] : p->eps_high;
    a.t_fix[l] = tfix ? tfix[layer0 + l] : p->t_fix;
  }
  a.withhold_tile = g_test_withhold_tile;
  a.wait_cycles = g_test_withhold_tile >= 0 ? g_test_wait_cycles : kK2WaitCycles;
  if (!mark(0)) return LASER_ERR_CUDA;
  if (a.T == 0) {
    // nothing to route: the call's offsets are all zero, loads and bins stay as they are (or
    // are this call's counts: zero)
    if (cudaMemsetAsync(a.offsets + (size_t)layer0 * (a.E + 1), 0,
                        sizeof(int32_t) * (size_t)n * (a.E + 1), s) != cudaSuccess)
      return LASER_ERR_CUDA;
    if (a.fresh &&
        (cudaMemsetAsync(a.loads + (size_t)layer0 * a.E, 0, sizeof(int32_t) * (size_t)n * a.E,
                         s) != cudaSuccess ||
         (a.bin_loads &&
          cudaMemsetAsync(a.bin_loads + (size_t)layer0 * a.n_bins, 0,
                          sizeof(int32_t) * (size_t)n * a.n_bins, s) != cudaSuccess)))
      return LASER_ERR_CUDA;
    return (mark(1) && mark(2) && mark(3)) ? LASER_OK : LASER_ERR_CUDA;
  }
  // clear the router's ready flags of these layers (one strided memset), then one launch for
  // the router and the ordered selection, one for the dispatch
  a.cluster_tiles = cluster_tiles_for(a, n);
  const size_t ready_bytes = sizeof(int32_t) * (size_t)((a.T + 15) / 16 + 2);
  if (a.cluster_tiles == 0 &&
      cudaMemset2DAsync(a.ws + (size_t)layer0 * a.ws_ls + a.lay.ready, a.ws_ls, 0, ready_bytes,
                        (size_t)n, s) != cudaSuccess)
    return LASER_ERR_CUDA;
  if (!mark(1)) return LASER_ERR_CUDA;
  if (launch_k12_for_E(a, n, s) != cudaSuccess) return LASER_ERR_CUDA;
  if (!mark(2)) return LASER_ERR_CUDA;
  if (a.fuse_dispatch) return mark(3) ? LASER_OK : LASER_ERR_CUDA;   // done by the selection blocks
  const int warps = k3_warps_per_block(a.E, a.k);
  const size_t smem3 = k3_block_smem_bytes(a.E) + (size_t)warps * k3_warp_smem_bytes(a.E, a.k);
  if (smem3 > 48 * 1024 &&
      cudaFuncSetAttribute(k3_dispatch, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem3) != cudaSuccess)
    return LASER_ERR_CUDA;
  dim3 g3((unsigned)((a.lay.n_groups + warps - 1) / warps), (unsigned)n);
  k3_dispatch<<<g3, warps * 32, smem3, s>>>(a);
  if (cudaGetLastError() != cudaSuccess) return LASER_ERR_CUDA;
  if (!mark(3)) return LASER_ERR_CUDA;
  return LASER_OK;
}

}  // namespace

extern "C" int laser_version(void) { return 200; }

extern "C" int laser_test_set_router(int mode) {
  if (mode != LASER_TEST_ROUTER_AUTO && mode != LASER_TEST_ROUTER_TILE &&
      mode != LASER_TEST_ROUTER_SPLITK && mode != LASER_TEST_ROUTER_TILE_ONESHOT)
    return -1;
  const int prev = g_test_router;
  g_test_router = mode;
  return prev;
}

namespace {
__global__ void k_empty() {}
}  // namespace

extern "C" int laser_test_launch_empty(void* cuda_stream) {
  k_empty<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>();
  return cudaGetLastError() == cudaSuccess ? 0 : -1;
}

extern "C" int laser_test_withhold_tile(int tile, long long wait_cycles) {
  if (tile >= 0 && wait_cycles < 1) return -1;
  g_test_withhold_tile = tile < 0 ? -1 : tile;
  g_test_wait_cycles = tile < 0 ? 0 : wait_cycles;
  return 0;
}

static_assert(kStatsWords == LASER_STATS_WORDS, "header and kernel disagree");

template <int N>
static void launch_stats(dim3 grid, cudaStream_t st, int T, int E, int k, const float* logits,
                         float near_ratio, int plateau_max, unsigned long long* stats) {
  k5_score_stats<N><<<grid, kStatsThreads, 0, st>>>(T, E, k, logits, near_ratio, plateau_max,
                                                    stats);
}

extern "C" int laser_score_stats(int32_t n_layers, int32_t T, int32_t E, int32_t k,
                                 const float* logits, float near_ratio, int32_t plateau_max,
                                 int32_t accumulate, int64_t* stats, float* means,
                                 void* cuda_stream) {
  if (n_layers < 1 || n_layers > 65535 || T < 0 || E < 1 || E > LASER_MAX_EXPERTS || k < 1 ||
      k > E || !(near_ratio >= 0.0f && near_ratio <= 1.0f) || plateau_max < 1 || !stats ||
      (T > 0 && !logits) || (long long)T * n_layers >= (1ll << 30))
    return LASER_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  auto* acc = reinterpret_cast<unsigned long long*>(stats);
  if (!accumulate &&
      cudaMemsetAsync(stats, 0, sizeof(int64_t) * kStatsWords * (size_t)n_layers, st) !=
          cudaSuccess)
    return LASER_ERR_CUDA;
  if (T > 0) {
    // blocks of 32 tokens per pass; about four waves of blocks over all layers
    const int per_layer = (T + 31) / 32;
    int gx = (4 * 148 * 8 + n_layers - 1) / n_layers;
    if (per_layer <= 2 * gx) gx = per_layer;   // one pass each rather than an uneven second one
    const dim3 grid(gx < 1 ? 1 : gx, n_layers);
    if (E <= 8) launch_stats<8>(grid, st, T, E, k, logits, near_ratio, plateau_max, acc);
    else if (E <= 32) launch_stats<32>(grid, st, T, E, k, logits, near_ratio, plateau_max, acc);
    else if (E <= 64) launch_stats<64>(grid, st, T, E, k, logits, near_ratio, plateau_max, acc);
    else if (E <= 128) launch_stats<128>(grid, st, T, E, k, logits, near_ratio, plateau_max, acc);
    else launch_stats<256>(grid, st, T, E, k, logits, near_ratio, plateau_max, acc);
  }
  if (means) k5_stats_means<<<(n_layers + 127) / 128, 128, 0, st>>>(n_layers, acc, means);
  return cudaGetLastError() == cudaSuccess ? LASER_OK : LASER_ERR_CUDA;
}

extern "C" int laser_imbalance(int32_t n_layers, int32_t E, int32_t n_bins, const int32_t* offsets,
                               const int32_t* expert_to_bin, const float* placement,
                               float* imbalance, float* bin_imbalance, float* aggregate,
                               void* cuda_stream) {
  if (n_layers < 1 || n_layers > 65535 || E < 1 || E > LASER_MAX_EXPERTS || n_bins < 1 ||
      n_bins > (placement ? kK4MaxBins : E) || !offsets || !imbalance)
    return LASER_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  k4_imbalance<<<n_layers < 148 ? n_layers : 148, kK4Threads, 0, st>>>(
      n_layers, E, n_bins, offsets, expert_to_bin, placement, imbalance, bin_imbalance);
  if (aggregate)
    k4_aggregate<<<1, kK4Threads, 0, st>>>(n_layers, E, offsets, imbalance, bin_imbalance,
                                           aggregate);
  return cudaGetLastError() == cudaSuccess ? LASER_OK : LASER_ERR_CUDA;
}

extern "C" const char* laser_strerror(int status) {
  switch (status) {
    case LASER_OK: return "ok";
    case LASER_ERR_INVALID_ARG: return "invalid argument";
    case LASER_ERR_UNSUPPORTED: return "unsupported mode";
    case LASER_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case LASER_ERR_MISALIGNED: return "pointer or row stride not 16-byte aligned";
    case LASER_ERR_CUDA: return "CUDA runtime error";
    case LASER_ERR_STATIC_SCRATCH:
      return "parameters need more scratch than the library's built-in array holds";
    default: return "unknown status";
  }
}

extern "C" int laser_workspace_bytes(const laser_params* p, size_t* bytes) {
  if (!bytes) return LASER_ERR_INVALID_ARG;
  const int rc = validate_params(p);
  if (rc != LASER_OK) return rc;
  *bytes = make_layout(p->T, p->E, p->k, p->c).total;
  return LASER_OK;
}

extern "C" int laser_route_layers_profiled(
    int32_t n_layers, const void* hidden, const void* w_g, const float* bias, int32_t* loads,
    const int32_t* expert_to_bin, int32_t* bin_loads, const laser_params* p,
    const float* eps_high_per_layer, const float* t_fix_per_layer, int32_t* expert_ids,
    float* weights, int32_t* offsets, int32_t* perm, float* logits_out, int32_t* status_word,
    void* workspace, size_t workspace_bytes, void* cuda_stream, void* const* stage_events) {
  const int rc = validate_params(p);
  if (rc != LASER_OK) return rc;
  if (n_layers < 1) return LASER_ERR_INVALID_ARG;
  if (!w_g || !loads || !offsets || !workspace) return LASER_ERR_INVALID_ARG;
  if (p->T > 0 && (!hidden || !expert_ids || !weights || !perm)) return LASER_ERR_INVALID_ARG;
  if (!aligned16(hidden) || !aligned16(w_g)) return LASER_ERR_MISALIGNED;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return LASER_ERR_MISALIGNED;
  for (int l = 0; l < n_layers; ++l) {
    const float e = eps_high_per_layer ? eps_high_per_layer[l] : p->eps_high;
    const float t = t_fix_per_layer ? t_fix_per_layer[l] : p->t_fix;
    if (!(e >= 0.0f) || !(t >= 0.0f) || !(t <= 1.0f)) return LASER_ERR_INVALID_ARG;
  }
  const WorkspaceLayout lay = make_layout(p->T, p->E, p->k, p->c);
  if (workspace_bytes < lay.total * (size_t)n_layers) return LASER_ERR_WORKSPACE_TOO_SMALL;

  RouteArgs a;
  a.hidden = static_cast<const uint16_t*>(hidden);
  a.hidden_ls = (long long)p->T * p->ld_hidden;
  a.wg = static_cast<const uint16_t*>(w_g);
  a.wg_ls = (long long)p->E * p->ld_w;
  a.bias = bias;
  a.loads = loads;
  a.e2b = expert_to_bin;
  a.bin_loads = bin_loads;
  a.fresh = p->fresh_loads != 0;
  a.expert_ids = expert_ids;
  a.weights = weights;
  a.offsets = offsets;
  a.perm = perm;
  a.logits_out = logits_out;
  a.status = status_word;
  a.ws = static_cast<unsigned char*>(workspace);
  a.ws_ls = lay.total;
  a.lay = lay;
  a.T = p->T; a.d = p->d; a.E = p->E; a.k = p->k; a.c = p->c;
  a.n_bins = p->n_bins; a.renorm = p->renormalize ? 1 : 0;
  a.G = p->update_granularity;
  a.fuse_dispatch = a.lay.n_groups <= kFusedDispatchGroups ? 1 : 0;
  a.trim_random = p->trim_mode == 1 ? 1 : 0;
  a.seed = p->seed;
  a.ld_h = p->ld_hidden; a.ld_w = p->ld_w;

  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  for (int l0 = 0; l0 < n_layers; l0 += kMaxLayersPerLaunch) {
    const int n = n_layers - l0 < kMaxLayersPerLaunch ? n_layers - l0 : kMaxLayersPerLaunch;
    const int r = enqueue_group(a, l0, n, p, eps_high_per_layer, t_fix_per_layer, s, stage_events);
    if (r != LASER_OK) return r;
  }
  return LASER_OK;
}

extern "C" int laser_route_layers(int32_t n_layers, const void* hidden, const void* w_g,
                                  const float* bias, int32_t* loads,
                                  const int32_t* expert_to_bin, int32_t* bin_loads,
                                  const laser_params* p, const float* eps_high_per_layer,
                                  const float* t_fix_per_layer, int32_t* expert_ids,
                                  float* weights, int32_t* offsets, int32_t* perm,
                                  float* logits_out, int32_t* status_word, void* workspace,
                                  size_t workspace_bytes, void* cuda_stream) {
  return laser_route_layers_profiled(n_layers, hidden, w_g, bias, loads, expert_to_bin, bin_loads,
                                     p, eps_high_per_layer, t_fix_per_layer, expert_ids, weights,
                                     offsets, perm, logits_out, status_word, workspace,
                                     workspace_bytes, cuda_stream, nullptr);
}

extern "C" int laser_route(const void* hidden, const void* w_g, const float* bias, int32_t* loads,
                           const int32_t* expert_to_bin, int32_t* bin_loads,
                           const laser_params* p, int32_t* expert_ids, float* weights,
                           int32_t* offsets, int32_t* perm, float* logits_out,
                           int32_t* status_word, void* workspace, size_t workspace_bytes,
                           void* cuda_stream) {
  return laser_route_layers(1, hidden, w_g, bias, loads, expert_to_bin, bin_loads, p, nullptr,
                            nullptr, expert_ids, weights, offsets, perm, logits_out, status_word,
                            workspace, workspace_bytes, cuda_stream);
}

namespace {
struct HostArena {
  size_t hidden, wg, bias, loads, e2b, bins, ids, weights, offsets, perm, status, ws, total;
};
HostArena make_arena(int L, const laser_params* p) {
  HostArena h;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align256(off + bytes); return o; };
  h.hidden = take(2ull * L * p->T * p->ld_hidden);
  h.wg = take(2ull * L * p->E * p->ld_w);
  h.bias = take(4ull * L * p->E);
  h.loads = take(4ull * L * p->E);
  h.e2b = take(4ull * p->E);
  h.bins = take(4ull * L * p->n_bins);
  h.ids = take(4ull * L * p->T * p->k);
  h.weights = take(4ull * L * p->T * p->k);
  h.offsets = take(4ull * L * (p->E + 1));
  h.perm = take(4ull * L * p->T * p->k);
  h.status = take(4);
  h.ws = take(make_layout(p->T, p->E, p->k, p->c).total * (size_t)L);
  h.total = off;
  return h;
}
}  // namespace

extern "C" int laser_host_arena_bytes(int32_t n_layers, const laser_params* p, size_t* bytes) {
  if (!bytes || n_layers < 1) return LASER_ERR_INVALID_ARG;
  const int rc = validate_params(p);
  if (rc != LASER_OK) return rc;
  *bytes = make_arena(n_layers, p).total;
  return LASER_OK;
}

extern "C" int laser_route_host(int32_t n_layers, const void* hidden, const void* w_g,
                                const float* bias, int32_t* loads, const int32_t* expert_to_bin,
                                int32_t* bin_loads, const laser_params* p,
                                const float* eps_high_per_layer, const float* t_fix_per_layer,
                                int32_t* expert_ids, float* weights, int32_t* offsets,
                                int32_t* perm, int32_t* status_out, void* arena,
                                size_t arena_bytes, void* cuda_stream) {
  const int rc = validate_params(p);
  if (rc != LASER_OK) return rc;
  if (n_layers < 1 || !arena || !w_g || !loads || !offsets) return LASER_ERR_INVALID_ARG;
  if (p->T > 0 && (!hidden || !expert_ids || !weights || !perm)) return LASER_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return LASER_ERR_MISALIGNED;
  const HostArena h = make_arena(n_layers, p);
  if (arena_bytes < h.total) return LASER_ERR_WORKSPACE_TOO_SMALL;
  unsigned char* base = static_cast<unsigned char*>(arena);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const size_t L = (size_t)n_layers, T = (size_t)p->T, E = (size_t)p->E, k = (size_t)p->k;
#define LASER_COPY(dst, src, bytes, kind)                                             \
  do {                                                                                \
    if ((bytes) > 0 && cudaMemcpyAsync((dst), (src), (bytes), (kind), s) != cudaSuccess) \
      return LASER_ERR_CUDA;                                                          \
  } while (0)
  LASER_COPY(base + h.hidden, hidden, 2 * L * T * p->ld_hidden, cudaMemcpyHostToDevice);
  LASER_COPY(base + h.wg, w_g, 2 * L * E * p->ld_w, cudaMemcpyHostToDevice);
  if (bias) LASER_COPY(base + h.bias, bias, 4 * L * E, cudaMemcpyHostToDevice);
  LASER_COPY(base + h.loads, loads, 4 * L * E, cudaMemcpyHostToDevice);
  if (expert_to_bin) LASER_COPY(base + h.e2b, expert_to_bin, 4 * E, cudaMemcpyHostToDevice);
  if (bin_loads) LASER_COPY(base + h.bins, bin_loads, 4 * L * p->n_bins, cudaMemcpyHostToDevice);
  if (cudaMemsetAsync(base + h.status, 0, 4, s) != cudaSuccess) return LASER_ERR_CUDA;

  const int r = laser_route_layers(
      n_layers, base + h.hidden, base + h.wg, bias ? reinterpret_cast<float*>(base + h.bias) : nullptr,
      reinterpret_cast<int32_t*>(base + h.loads),
      expert_to_bin ? reinterpret_cast<int32_t*>(base + h.e2b) : nullptr,
      bin_loads ? reinterpret_cast<int32_t*>(base + h.bins) : nullptr, p, eps_high_per_layer,
      t_fix_per_layer, reinterpret_cast<int32_t*>(base + h.ids),
      reinterpret_cast<float*>(base + h.weights), reinterpret_cast<int32_t*>(base + h.offsets),
      reinterpret_cast<int32_t*>(base + h.perm), nullptr,
      reinterpret_cast<int32_t*>(base + h.status), base + h.ws, h.total - h.ws, s);
  if (r != LASER_OK) return r;

  LASER_COPY(expert_ids, base + h.ids, 4 * L * T * k, cudaMemcpyDeviceToHost);
  LASER_COPY(weights, base + h.weights, 4 * L * T * k, cudaMemcpyDeviceToHost);
  LASER_COPY(offsets, base + h.offsets, 4 * L * (E + 1), cudaMemcpyDeviceToHost);
  LASER_COPY(perm, base + h.perm, 4 * L * T * k, cudaMemcpyDeviceToHost);
  LASER_COPY(loads, base + h.loads, 4 * L * E, cudaMemcpyDeviceToHost);
  if (bin_loads) LASER_COPY(bin_loads, base + h.bins, 4 * L * p->n_bins, cudaMemcpyDeviceToHost);
  if (status_out) LASER_COPY(status_out, base + h.status, 4, cudaMemcpyDeviceToHost);
#undef LASER_COPY
  if (cudaStreamSynchronize(s) != cudaSuccess) return LASER_ERR_CUDA;
  return LASER_OK;
}
