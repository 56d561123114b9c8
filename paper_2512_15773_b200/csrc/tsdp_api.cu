// libtsdp: host side of the TS-DP speculative denoising loop -- context, weight loading, the round
// orchestration (plain launches or a captured CUDA graph per (B, K)) and the C ABI of include/tsdp.h.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <string>
#include <tuple>
#include <type_traits>
#include <utility>
#include <vector>

#include "../../include/tsdp.h"
#include "common.cuh"
#include "gemm_tcgen05.cuh"
#include "net_kernels.cuh"
#include "round_kernels.cuh"
#include "drafter_cluster.cuh"
#include "sched_kernel.cuh"
#include "dit_kernels.cuh"
#include "ctx_attn_tcgen05.cuh"
#include "unet_kernels.cuh"
#include "xattn_fold.cuh"
#include "draft_tail.cuh"
#include "distill_kernels.cuh"

using namespace tsdp;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct XfmrLayer {
  float *ln1_g, *ln1_b, *bqkv, *bo, *ln2_g, *ln2_b, *bq2, *bo2, *ln3_g, *ln3_b, *b1, *b2;
  void *Wqkv, *Wo, *Wq2, *Wo2, *W1, *W2;      // [out, in], bf16 or fp32 by precision
  // decoder transformer, bf16, 64-wide heads, H = 16: the QKV projection again with its output features ordered
  // head by head, [Q_h | K_h | V_h] (64 each), for the GEMM whose epilogue runs the self-attention (null: not built)
  void* Wqkv_hm = nullptr;
  float* bqkv_hm = nullptr;
};

struct Net {
  tsdp_net_t cfg{};
  bool loaded = false;
  float m0 = 0.f, s0 = 1.f;                   // GAUSS
  MlpWeights mlp{};                           // MLP
  float *W_in = nullptr, *b_in = nullptr, *pos = nullptr, *W_obs = nullptr, *b_obs = nullptr, *cpos = nullptr;
  float *lnf_g = nullptr, *lnf_b = nullptr, *W_outT = nullptr, *b_out = nullptr;
  std::vector<XfmrLayer> L;
  void* Wkv_all = nullptr;                    // [L*2d, d]: the cross-attention K/V projections of all blocks
  float* bkv_all = nullptr;
  float* kv_time = nullptr;                   // [T, L*2d]   K/V of the time token for every timestep
  float* kv_obs = nullptr;                    // [max_B*To, L*2d]  K/V of the obs tokens, per chunk
  float* temb_table = nullptr;                // [T, temb or d] sinusoidal embedding
  // XFMR, bf16: cross-attention folded into the memory tokens (xattn_fold.cuh); tables per timestep / per request token
  bool fold = false;
  XfoldLayerW* fold_lw = nullptr;             // [L] device
  __nv_bfloat16 *fold_kq_time = nullptr, *fold_ut_time = nullptr, *fold_kq_obs = nullptr, *fold_ut_obs = nullptr;
  float *fold_c_time = nullptr, *fold_c_obs = nullptr;
  float* mod = nullptr;                       // DIT: [T, L*6d + 2d] shift / scale / gate vectors of every timestep
  int mod_ld = 0;
  // UNET: residual blocks in execution order, FiLM tables, head
  struct UBlock { int cin, cout, foff; void *W1, *W2, *Wr; float *b1, *g1, *be1, *b2, *g2, *be2, *br; };
  std::vector<UBlock> ub;
  int F = 0;                                  // FiLM width: sum over blocks of 2 * cout
  float *film_time = nullptr, *film_obs = nullptr, *WfT_obs = nullptr, *obs_m = nullptr;   // [T,F], [items,F], [F,To*Do], [items,To*Do]
  void* Wh = nullptr;
  float *bh = nullptr, *gh = nullptr, *beh = nullptr;
  // UNET activations (zero-padded channels-last tensors, see unet_kernels.cuh), allocated at init
  struct UWs { void *X0 = nullptr, *E = nullptr, *M1 = nullptr, *M2 = nullptr, *HB = nullptr;
               void *TMP[4] = {}, *D[4] = {}, *CAT[4] = {}, *P[4] = {}, *U1[4] = {}, *U2[4] = {};
               float *Y = nullptr, *R = nullptr; size_t Y_cap = 0; } uw;
  std::vector<void*> allocs;
};

}  // namespace

struct tsdp_ctx {
  tsdp_config_t cfg{};
  int D = 0, num_sms = 148;
  Net net[2];
  DdpmTables S{};
  std::vector<void*> allocs;
  // round state
  float *xt = nullptr, *muhat = nullptr, *eps = nullptr, *eps_d = nullptr, *actions = nullptr, *obs = nullptr;
  int* t = nullptr;
  // continuous batching: slot -> request it serves, next waiting request, number of requests, capacity of the
  // per-request buffers (obs, actions, obs K/V, scheduler outputs)
  int *item = nullptr, *queue_head = nullptr, *n_items = nullptr;
  size_t items_cap = 0;
  uint64_t* seed = nullptr;
  int *round_idx = nullptr, *n_done = nullptr, *status = nullptr;
  int* host_done = nullptr;                   // mapped pinned
  RoundParams* sched = nullptr;               // device, capacity TSDP_MAX_T + 1
  RoundParams* sched_host = nullptr;          // pinned staging
  DevStats* stats = nullptr;
  float* dbg_logalpha = nullptr;
  int* dbg_jstar = nullptr;
  // transformer workspaces (bytes sized for the larger of the two nets)
  float* h = nullptr;
  void *a = nullptr, *qkv = nullptr, *q2 = nullptr, *f = nullptr, *memtok = nullptr;
  // schedule set by the caller
  std::vector<int> sched_K;
  std::vector<tsdp_accept_t> sched_acc;
  // graphs and tensor maps
  struct GraphRec { cudaGraphExec_t exec; int launches; };
  std::map<std::tuple<int, int>, GraphRec> graphs;
  std::map<std::tuple<const void*, int, int, int, int, int, int>, CUtensorMap> maps;
  std::map<void*, size_t> guards;             // device buffer -> its size: the guard bytes sit right behind it
  EncodeTiledFn encode = nullptr;
  cudaStream_t cap_stream = nullptr;
  // persistent cluster drafter: usable for this configuration, shared memory per CTA, clusters that fit the GPU
  // scheduler network (Sec. 3.3): weights, per-environment outputs, its inputs, the side stream it runs on
  SchedWeights sched_w{};
  bool sched_loaded = false, sched_on = false;
  EnvParams* envp = nullptr;
  float *progress = nullptr, *sched_dbg = nullptr;
  int* item_counts = nullptr;        // per request: drafts proposed, drafts accepted, rounds, reverse steps taken
  float* reward = nullptr;
  float *distill_theta = nullptr, *distill_terms = nullptr;   // Gaussian-drafter distillation step: (m0, s0), per-sample terms
  double* distill_res = nullptr;
  int items_last = 0;                // requests of the last chunk call
  std::vector<void*> sched_allocs;
  cudaStream_t side_stream = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  // second stream of a forward: the 1x1 residual convolution of a UNet block runs beside the block's two kernel-5
  // convolutions (it only needs the block's input) and joins in front of the block's last GroupNorm
  cudaStream_t aux_stream = nullptr;
  cudaEvent_t ev_aux_fork = nullptr, ev_aux_join = nullptr;
  bool aux_on = true;                          // TSDP_NO_AUX_STREAM: everything on one stream
  // device time of the last chunk calls (ring buffer behind the latency percentiles of tsdp_stats)
  cudaEvent_t ev_chunk0 = nullptr, ev_chunk1 = nullptr;
  std::vector<float> lat_ring;
  size_t lat_pos = 0, lat_n = 0;
  bool pdl = true;                            // programmatic dependent launch between the kernels of a round
  int tc_attn = 1;                            // context cross-attention on tcgen05: 0 never (TSDP_NO_TC_ATTN), 1 large groups, 2 always (TSDP_TC_ATTN=2)
  bool async_bcast = true;                    // cluster kernel: st.async + mbarrier stage hand-over (TSDP_NO_ASYNC_BCAST unset)
  bool dc_ok = false;
  bool no_ksplit = false;                      // TSDP_NO_KSPLIT: convolution GEMMs never split their reduction
  int dc_smem = 0, dc_max_clusters = 0;
  bool dc_resident = false;
  // the same cluster kernel running the BASE model's verification forward (small batches of small transformers)
  bool cv_ok = false, cv_resident = false;
  int cv_smem = 0, cv_max_clusters = 0;
  uint64_t rounds = 0, launches = 0;
  int launches_per_round_tmp = 0;
  // plan of a round (round_plan_kernel): compacted candidate list of the verification forward, slot order and
  // per-step counts of the drafter; `compact` off: every forward runs on the dense B x (K+1) layout
  bool compact = true;
  int *plan_live_n = nullptr, *plan_list = nullptr, *plan_slot_start = nullptr, *plan_order = nullptr, *plan_dn = nullptr;
  // live-row information of the forward pass being enqueued (set by forward(), read by the launch helpers)
  const int* live_n = nullptr;
  const int* live_slot_start = nullptr;
  int live_static = 0;
  // while profiling: host copies of the plan's counts, so that a GEMM's flops are those of the rows it really processed
  int prof_plan_live = -1, prof_plan_dn[TSDP_MAX_K + 2] = {};
  int prof_live_count = -1;                   // live candidates of the forward being enqueued (-1: unknown, use the dense count)
  // CTA-pair GEMM (cta_group::2): clusters of two CTAs that fit the device at once (0: not usable), and whether it is used
  int pair_clusters = 0, pair_clusters_attn = 0;
  int pair_mode = 1;                          // TSDP_GEMM_PAIR: 0 never, 1 (default) by shape (use_pair_gemm), 2 wherever it applies
  bool dbg_armed = false, dbg_in_test_gemm = false;   // tsdp_debug_arm_gemm_timeout
  long long dbg_wait_cycles = 0;
  uint64_t cand_static = 0;                   // candidates the dense layout would have evaluated since the last reset
  // optional per-kernel-family timing with CUDA events (plain launches, no graph)
  bool prof_on = false;
  int prof_gemm_cat = 0;                      // 0 while the base model runs, 6 while the drafter runs
  int force_bn = 0;                           // TSDP_GEMM_BN
  bool xf_skip_embed = false, xf_skip_head = false;   // layer-by-layer drafter: draft_tail_kernel does those parts
  std::vector<cudaEvent_t> prof_ev;
  std::vector<int> prof_cat;
  std::vector<double> prof_flop;
  std::string last_error;
};

namespace {

#define CU_TRY(ctx, expr)                                                                         \
  do {                                                                                            \
    cudaError_t e__ = (expr);                                                                     \
    if (e__ != cudaSuccess) {                                                                     \
      (ctx)->last_error = std::string(#expr) + ": " + cudaGetErrorString(e__);                    \
      return TSDP_ERR_CUDA;                                                                       \
    }                                                                                             \
  } while (0)

// Every device buffer of a context is followed by a 256-byte guard filled with a pattern; tsdp_debug_check_guards
// verifies that no kernel wrote past a buffer's end (the stand-in for a memory checker on the kernels' index math).
constexpr size_t GUARD_BYTES = 256;
constexpr int GUARD_PATTERN = 0xA5;

template <typename T>
int dev_alloc(tsdp_ctx* c, std::vector<void*>& pool, T** p, size_t n) {
  void* q = nullptr;
  const size_t bytes = (n * sizeof(T) + 15) / 16 * 16;
  CU_TRY(c, cudaMalloc(&q, bytes + GUARD_BYTES));
  CU_TRY(c, cudaMemset(q, 0, bytes));
  CU_TRY(c, cudaMemset(static_cast<uint8_t*>(q) + bytes, GUARD_PATTERN, GUARD_BYTES));
  pool.push_back(q);
  c->guards[q] = bytes;
  *p = reinterpret_cast<T*>(q);
  return TSDP_OK;
}
void dev_free_pool(tsdp_ctx* c, std::vector<void*>& pool) {
  for (void* q : pool) { c->guards.erase(q); cudaFree(q); }
  pool.clear();
}

int alloc_bytes(tsdp_ctx* c, std::vector<void*>& pool, void** p, size_t bytes) {
  return dev_alloc<uint8_t>(c, pool, reinterpret_cast<uint8_t**>(p), bytes);
}

// Every kernel of the round is launched with programmatic stream serialisation: the next kernel of the
// chain may be scheduled and run its prologue while this one drains; each kernel calls pdl_wait()
// (griddepcontrol.wait) before it touches memory that its predecessors write or read.
template <typename... P, typename... A>
void launch_kernel(tsdp_ctx* c, void (*kern)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, A&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = c->pdl ? 1 : 0;
  cudaLaunchKernelEx(&cfg, kern, std::forward<A>(args)...);   // a failure is read by cudaGetLastError at the call site
}
// The same for a kernel that runs in clusters of `cluster` CTAs along x.
template <typename... P, typename... A>
void launch_kernel_cluster(tsdp_ctx* c, void (*kern)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, int cluster, A&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = cluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = c->pdl ? 2 : 1;
  cudaLaunchKernelEx(&cfg, kern, std::forward<A>(args)...);
}
#define TSDP_LAUNCH(ctx, kern, grid, block, smem, stream, ...) \
  launch_kernel(ctx, kern, dim3(grid), dim3(block), (size_t)(smem), stream, __VA_ARGS__)

constexpr size_t PROF_CAP = 60000;
void prof_begin(tsdp_ctx* c, cudaStream_t s, int cat, double flop) {
  if (!c->prof_on || c->prof_cat.size() >= PROF_CAP) return;
  if (c->prof_gemm_cat == 6 && cat >= 1 && cat <= 3) cat += 9;      // the drafter's LayerNorm / attention / embedding-head kernels
  cudaEvent_t a, b;
  if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return;
  c->prof_ev.push_back(a); c->prof_ev.push_back(b);
  c->prof_cat.push_back(cat); c->prof_flop.push_back(flop);
  cudaEventRecord(a, s);
}
void prof_end(tsdp_ctx* c, cudaStream_t s) {
  if (!c->prof_on || c->prof_ev.empty() || c->prof_ev.size() != 2 * c->prof_cat.size()) return;
  cudaEventRecord(c->prof_ev.back(), s);
}

// Live-row descriptor for a kernel whose launch was sized for `per` rows per candidate of the current forward.
LiveRows live_desc(const tsdp_ctx* c, int per, int add = 0) { return LiveRows{c->live_n, per, add}; }

// (C_in, C_out) of the residual blocks of the conv UNet in execution order: two per level down, two in the
// middle, two per level up (the first of which takes the concatenation [upsampled | skip]).
std::vector<std::pair<int, int>> unet_channels(int c, int levels) {
  std::vector<std::pair<int, int>> out;
  int cin = c;
  for (int lv = 0; lv < levels; ++lv) { out.push_back({cin, c << lv}); out.push_back({c << lv, c << lv}); cin = c << lv; }
  out.push_back({cin, cin}); out.push_back({cin, cin});
  for (int lv = levels - 2; lv >= 0; --lv) { out.push_back({cin + (c << lv), c << lv}); out.push_back({c << lv, c << lv}); cin = c << lv; }
  return out;
}

bool net_cfg_ok(const tsdp_config_t& cfg, const tsdp_net_t& n) {
  if (n.arch == TSDP_ARCH_GAUSS) return true;
  if (n.arch == TSDP_ARCH_FROZEN) return &n == &cfg.draft;      // a way to draft, not a network: drafter only
  if (n.arch == TSDP_ARCH_MLP)
    return n.layers >= 1 && n.layers <= MLP_MAX_LAYERS && n.d >= 1 && n.d <= 4096 && n.temb >= 2 && n.temb % 2 == 0;
  if (n.arch == TSDP_ARCH_XFMR)
    return n.layers >= 1 && n.d % 128 == 0 && n.d >= 128 && n.d <= 1024 && n.heads >= 1 && n.d % n.heads == 0 &&
           (n.d / n.heads) % 32 == 0 && (n.d / n.heads) <= 128 && cfg.H <= 64 && cfg.obs_tokens <= 8 && cfg.A <= 64;
  if (n.arch == TSDP_ARCH_UNET)
    return n.layers >= 1 && n.layers <= 4 && n.d % 128 == 0 && n.d >= 128 && (n.d << (n.layers - 1)) <= 2048 && n.heads >= 1 &&
           n.d % n.heads == 0 && n.temb >= 4 && n.temb % 4 == 0 && cfg.H % (1 << (n.layers - 1)) == 0 && cfg.H <= 64 &&
           cfg.A <= 64;
  if (n.arch == TSDP_ARCH_DIT)
    return n.layers >= 1 && n.d % 128 == 0 && n.d >= 128 && n.d <= 1024 && n.heads >= 1 && n.d % n.heads == 0 &&
           (n.d / n.heads) % 32 == 0 && (n.d / n.heads) <= 128 && cfg.H <= 64 && cfg.obs_tokens >= 1 &&
           cfg.obs_tokens <= 256 && cfg.obs_dim >= 1 && cfg.A <= 64;
  return false;
}

size_t weights_count(const tsdp_config_t& cfg, const tsdp_net_t& n) {
  const size_t D = (size_t)cfg.H * cfg.A, d = n.d;
  if (n.arch == TSDP_ARCH_GAUSS) return 2;
  if (n.arch == TSDP_ARCH_MLP) {
    size_t in = D + n.temb + (size_t)cfg.obs_tokens * cfg.obs_dim, tot = 0;
    for (int l = 0; l < n.layers; ++l) { tot += in * d + d; in = d; }
    return tot + in * D + D;
  }
  if (n.arch == TSDP_ARCH_XFMR) {
    size_t tot = (size_t)cfg.A * d + d + (size_t)cfg.H * d + (size_t)cfg.obs_dim * d + d + (size_t)(1 + cfg.obs_tokens) * d;
    const size_t per = 2 * d + d * 3 * d + 3 * d + d * d + d + 2 * d + d * d + d + d * 2 * d + 2 * d + d * d + d + 2 * d +
                       d * 4 * d + 4 * d + 4 * d * d + d;
    return tot + per * n.layers + 2 * d + d * cfg.A + cfg.A;
  }
  if (n.arch == TSDP_ARCH_UNET) {
    const size_t dt = n.temb, dc = dt + (size_t)cfg.obs_tokens * cfg.obs_dim;
    size_t tot = (size_t)cfg.A * d + d + dt * 4 * dt + 4 * dt + 4 * dt * dt + dt;
    for (auto& cc : unet_channels((int)d, n.layers)) {
      const size_t ci = cc.first, co = cc.second;
      tot += 5 * ci * co + co + 2 * co + dc * 2 * co + 2 * co + 5 * co * co + co + 2 * co + (ci != co ? ci * co + co : 0);
    }
    return tot + 5 * d * d + d + 2 * d + d * cfg.A + cfg.A;
  }
  if (n.arch == TSDP_ARCH_DIT) {
    size_t tot = (size_t)cfg.A * d + d + (size_t)cfg.H * d + (size_t)cfg.obs_dim * d + d + (size_t)cfg.obs_tokens * d +
                 2 * (d * d + d);
    const size_t per = d * 6 * d + 6 * d + d * 3 * d + 3 * d + d * d + d + 2 * d + d * d + d + d * 2 * d + 2 * d + d * d + d +
                       d * 4 * d + 4 * d + 4 * d * d + d;
    return tot + per * n.layers + d * 2 * d + 2 * d + d * cfg.A + cfg.A;
  }
  return 0;
}

size_t sched_weights_count(const tsdp_config_t& cfg) {
  const size_t obs_len = (size_t)cfg.obs_tokens * cfg.obs_dim, D = (size_t)cfg.H * cfg.A;
  return obs_len * SCHED_HID + SCHED_HID + D * SCHED_HID + SCHED_HID + SCHED_PROG + SCHED_PROG +
         (size_t)SCHED_CAT * SCHED_HID + SCHED_HID + (size_t)SCHED_HID * SCHED_OUT + SCHED_OUT;
}

// ------------------------------------------------------------------------------------------ GEMM
// Tiled 2-D tensor map with the 128-byte swizzle over a row-major [rows, cols] matrix whose rows are
// `ld` elements apart; esz = 2 (bf16) or 4 (fp32).  The box is box_cols x box_rows (box_cols * esz = 128).
int get_map(tsdp_ctx* c, const void* ptr, int esz, int rows, int cols, int ld, int box_cols, int box_rows,
            CUtensorMap* out) {
  auto key = std::make_tuple(ptr, esz, rows, cols, ld, box_cols, box_rows);
  auto it = c->maps.find(key);
  if (it != c->maps.end()) { *out = it->second; return TSDP_OK; }
  CUtensorMap m;
  cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t gstr[1] = {(cuuint64_t)ld * esz};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = c->encode(&m, esz == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                         const_cast<void*>(ptr), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    c->last_error = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r);
    return TSDP_ERR_CUDA;
  }
  c->maps[key] = m;
  *out = m;
  return TSDP_OK;
}

// Rows a GEMM of the forward being enqueued really processes, as far as the host knows (profiling mode reads the
// round's plan back); otherwise the dense count.
int gemm_rows_known(const tsdp_ctx* c, const GemmArgs& g) {
  if (g.live.n == nullptr || c->prof_live_count < 0) return g.M;
  const int v = c->prof_live_count * g.live.mul + g.live.add;
  return v < 0 ? 0 : (v < g.M ? v : g.M);
}

template <int BN, int EPI>
int launch_tc(tsdp_ctx* c, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const GemmArgs& g,
              cudaStream_t s) {
  const int tiles = ((g.M + GEMM_BM - 1) / GEMM_BM) * (g.N / BN) * (g.ksplit > 1 ? g.ksplit : 1);
  const int grid = tiles < c->num_sms ? tiles : c->num_sms;
  prof_begin(c, s, c->prof_gemm_cat, 2.0 * gemm_rows_known(c, g) * g.N * g.K);
  TSDP_LAUNCH(c, (gemm_tcgen05_kernel<BN, EPI>), grid, GEMM_THREADS, gemm_smem_bytes(BN), s, ma, mb, mc, g);
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

// 256 x 256 tiles on CTA pairs (cta_group::2); `mb` is the W map with a box of 128 rows (each CTA stages half a tile).
template <int EPI>
int launch_tc_pair(tsdp_ctx* c, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const GemmArgs& g,
                   cudaStream_t s) {
  const int tiles = ((g.M + 2 * GEMM_BM - 1) / (2 * GEMM_BM)) * (g.N / 256);
  const int pairs = tiles < c->pair_clusters ? tiles : c->pair_clusters;
  prof_begin(c, s, c->prof_gemm_cat, 2.0 * gemm_rows_known(c, g) * g.N * g.K);
  launch_kernel_cluster(c, gemm_tcgen05_kernel<256, EPI, 2>, dim3(2 * pairs), dim3(GEMM_THREADS), (size_t)gemm_smem_bytes_cg(256, 2), s, 2,
                        ma, mb, mc, g);
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}
int launch_tc_pair_epi(tsdp_ctx* c, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const GemmArgs& g,
                       int epi, cudaStream_t s) {
  switch (epi) {
    case EPI_STORE: return launch_tc_pair<EPI_STORE>(c, ma, mb, mc, g, s);
    case EPI_GELU: return launch_tc_pair<EPI_GELU>(c, ma, mb, mc, g, s);
    case EPI_RESID: return launch_tc_pair<EPI_RESID>(c, ma, mb, mc, g, s);
    case EPI_GATE: return launch_tc_pair<EPI_GATE>(c, ma, mb, mc, g, s);
    default: return launch_tc_pair<EPI_F32>(c, ma, mb, mc, g, s);
  }
}
// Whether a GEMM runs on CTA pairs: wide outputs, enough 256 x 256 tiles to occupy the pairs, and a long reduction.
// Measured (45 056 - 54 400 rows): with K >= 1024 the pair form is 5 - 12 % faster on every shape (1.28 -> 1.43 PFLOP/s
// at N 3072, K 1024); at K = 512 a tile has only 8 k-blocks, the epilogue and the hand-overs weigh as much as the
// mainloop, and the two forms tie or the single-CTA one wins by a few per cent.
bool use_pair_gemm(const tsdp_ctx* c, int M, int N, int K) {
  if (c->pair_mode == 0 || c->pair_clusters < 1 || N % 256 != 0) return false;
  if (c->pair_mode == 2) return true;
  const long long tiles = (long long)((M + 255) / 256) * (N / 256);
  return K >= 1024 && tiles * 5 >= (long long)c->pair_clusters * 4;
}

template <int BN>
int launch_tc_epi(tsdp_ctx* c, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const GemmArgs& g,
                  int epi, cudaStream_t s) {
  switch (epi) {
    case EPI_STORE: return launch_tc<BN, EPI_STORE>(c, ma, mb, mc, g, s);
    case EPI_GELU: return launch_tc<BN, EPI_GELU>(c, ma, mb, mc, g, s);
    case EPI_RESID: return launch_tc<BN, EPI_RESID>(c, ma, mb, mc, g, s);
    case EPI_GATE: return launch_tc<BN, EPI_GATE>(c, ma, mb, mc, g, s);
    default: return launch_tc<BN, EPI_F32>(c, ma, mb, mc, g, s);
  }
}

template <int BN, int EPI>
cudaError_t set_smem_attr() {
  return cudaFuncSetAttribute(gemm_tcgen05_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              gemm_smem_bytes(BN));
}
template <int BN>
cudaError_t set_smem_attr_all() {
  cudaError_t e;
  if ((e = set_smem_attr<BN, EPI_STORE>()) != cudaSuccess) return e;
  if ((e = set_smem_attr<BN, EPI_GELU>()) != cudaSuccess) return e;
  if ((e = set_smem_attr<BN, EPI_RESID>()) != cudaSuccess) return e;
  if ((e = set_smem_attr<BN, EPI_GATE>()) != cudaSuccess) return e;
  return set_smem_attr<BN, EPI_F32>();
}

// Tile width: the widest BN in {256, 128, 64, 32} dividing N whose tiles still fill 60 % of the SMs, else the
// narrowest that divides N (small-batch calls are latency-bound and want many CTAs).  Measured on the block's
// shapes at 4 k - 45 k rows: per flop a 128-wide tile costs 1.24x and a 64-wide one 2.15x of a 256-wide one (the
// k-loop of a narrow tile is bound by loading the 128-row A block, which does not shrink), so a wide tile that
// leaves a third of the SMs idle still beats two waves of narrow ones; below about half occupancy it does not.
int pick_bn(int M, int N, int num_sms) {
  const int tm = (M + GEMM_BM - 1) / GEMM_BM;
  const int cands[4] = {256, 128, 64, 32};
  for (int i = 0; i < 4; ++i)
    if (N % cands[i] == 0 && (long long)tm * (N / cands[i]) * 5 >= (long long)num_sms * 3) return cands[i];
  for (int i = 3; i >= 0; --i)
    if (N % cands[i] == 0) return cands[i];
  return 0;
}

// Parts into which the reduction of a convolution GEMM [M x N x K] -> fp32 is split (1: not at all).  With a small batch
// the deep levels of the UNet are a handful of narrow tiles (16 - 32 CTAs) that each walk 80 - 160 k-blocks one after the
// other: cutting the k range puts those k-blocks on otherwise idle SMs, each part writes its partial sums to a buffer
// of its own and the GroupNorm kernel that consumes them adds the parts in order (same bits whatever ran where; a
// function of the launch shape only).  Parts of at least 4 k-blocks, at most 8 parts, no more units than SMs, and
// only where the tiles use the plain-store epilogue (widths below 128).
int conv_ksplit(const tsdp_ctx* c, int M, int N, int K, size_t cap_elems) {
  if (c->no_ksplit || c->cfg.precision == 0 || M <= 0 || K % GEMM_BK != 0 || N % 32 != 0) return 1;
  if (c->force_bn == 0 && use_pair_gemm(c, M, N, K)) return 1;
  const int BN = (c->force_bn > 0 && N % c->force_bn == 0) ? c->force_bn : pick_bn(M, N, c->num_sms);
  if (gemm_tma_epilogue(BN)) return 1;
  const int tiles = ((M + GEMM_BM - 1) / GEMM_BM) * (N / BN), kblocks = K / GEMM_BK;
  int S = 1;
  while (S < 8 && tiles * S * 2 <= c->num_sms && kblocks / (S * 2) >= 4 && (size_t)(S * 2) * (size_t)(M + 4) * (size_t)N <= cap_elems) S *= 2;
  return S;
}

// Gate of an adaptive-LayerNorm residual (EPI_GATE): gate vectors and the row -> timestep map.
struct GateSpec {
  const float* gate; int gate_ld; const CandMap* cm; int H, Tsteps;
};

int gemm(tsdp_ctx* c, const void* A, const void* W, const float* bias, int M, int N, int K, int epi, void* out,
         int ldo, cudaStream_t s, const GateSpec* gs = nullptr, int conv_c = 0, int ksplit = 1, long long split_stride = 0) {
  if (M <= 0) return TSDP_OK;
  GemmArgs g{M, N, K, bias, out, ldo, c->status, nullptr, 0, nullptr, 1, 0, 1, 1, conv_c > 0 ? conv_c : K, conv_c,
             LiveRows{nullptr, 0, 0}, nullptr, 0, 0, 0};
  if (c->dbg_armed && c->dbg_in_test_gemm && c->cfg.precision == 1) {      // one launch: see tsdp_debug_arm_gemm_timeout
    g.wait_cycles = c->dbg_wait_cycles;
    g.withhold_first_stage = 1;
    c->dbg_armed = false;
  }
  if (epi == EPI_GATE) {
    if (!gs) return TSDP_ERR_ARG;
    g.gate = gs->gate; g.gate_ld = gs->gate_ld; g.t = gs->cm->t; g.C = gs->cm->C; g.koff = gs->cm->koff; g.H = gs->H;
    g.Tsteps = gs->Tsteps; g.list = gs->cm->list;
  }
  if (c->live_n != nullptr && c->live_static > 0) {
    // rows per candidate of this GEMM: M = n rows_per (token rows), or n rows_per - 4 (a convolution over padded tensors)
    const int n = c->live_static;
    if (M % n == 0) g.live = LiveRows{c->live_n, M / n, 0};
    else if ((M + 4) % n == 0) g.live = LiveRows{c->live_n, (M + 4) / n, -4};
  }
  if (c->cfg.precision == 0) {
    dim3 grid((N + 63) / 64, (M + 63) / 64);
    const float* a = reinterpret_cast<const float*>(A);
    const float* w = reinterpret_cast<const float*>(W);
    prof_begin(c, s, c->prof_gemm_cat, 2.0 * gemm_rows_known(c, g) * N * K);
    switch (epi) {
      case EPI_GELU: TSDP_LAUNCH(c, (gemm_simt_kernel<EPI_GELU>), grid, 256, 0, s, a, w, g); break;
      case EPI_RESID: TSDP_LAUNCH(c, (gemm_simt_kernel<EPI_RESID>), grid, 256, 0, s, a, w, g); break;
      case EPI_GATE: TSDP_LAUNCH(c, (gemm_simt_kernel<EPI_GATE>), grid, 256, 0, s, a, w, g); break;
      default: TSDP_LAUNCH(c, (gemm_simt_kernel<EPI_F32>), grid, 256, 0, s, a, w, g); break;
    }
    prof_end(c, s);
    c->launches_per_round_tmp++;
    CU_TRY(c, cudaGetLastError());
    return TSDP_OK;
  }
  if (K % GEMM_BK != 0 || N % 32 != 0) {
    c->last_error = "tensor-core GEMM needs K % 64 == 0 and N % 32 == 0";
    return TSDP_ERR_ARG;
  }
  const bool pair = c->force_bn == 0 && use_pair_gemm(c, M, N, K);
  const int BN = pair ? 256 : ((c->force_bn > 0 && N % c->force_bn == 0) ? c->force_bn : pick_bn(M, N, c->num_sms));
  if (ksplit > 1) {      // see conv_ksplit: narrow tiles with the plain-store epilogue only
    if (pair || gemm_tma_epilogue(BN) || epi != EPI_F32 || ksplit > K / GEMM_BK) return TSDP_ERR_ARG;
    g.ksplit = ksplit; g.split_stride = split_stride;
  }
  CUtensorMap ma, mb, mc;
  int r;
  if (conv_c > 0) {      // kernel-5 convolution: A is the padded tensor [M + 4, conv_c] itself
    if (conv_c % GEMM_BK != 0 || K != 5 * conv_c) return TSDP_ERR_ARG;
    if ((r = get_map(c, A, 2, M + 4, conv_c, conv_c, GEMM_BK, GEMM_BM, &ma)) != TSDP_OK) return r;
  } else if ((r = get_map(c, A, 2, M, K, K, GEMM_BK, GEMM_BM, &ma)) != TSDP_OK) return r;
  if ((r = get_map(c, W, 2, N, K, K, GEMM_BK, pair ? BN / 2 : BN, &mb)) != TSDP_OK) return r;
  mc = ma;
  if (gemm_tma_epilogue(BN)) {   // the epilogue hands 128-row x 128-byte chunks to TMA
    const int esz = (epi == EPI_STORE || epi == EPI_GELU) ? 2 : 4;
    if (ldo % (16 / esz) != 0 || (reinterpret_cast<uintptr_t>(out) & 15) != 0) {
      c->last_error = "GEMM output must be 16-byte aligned with a row pitch that is a multiple of 16 bytes";
      return TSDP_ERR_ARG;
    }
    if ((r = get_map(c, out, esz, M, N, ldo, 128 / esz, GEMM_BM, &mc)) != TSDP_OK) return r;
  }
  if (pair) return launch_tc_pair_epi(c, ma, mb, mc, g, epi, s);
  switch (BN) {
    case 256: return launch_tc_epi<256>(c, ma, mb, mc, g, epi, s);
    case 128: return launch_tc_epi<128>(c, ma, mb, mc, g, epi, s);
    case 64: return launch_tc_epi<64>(c, ma, mb, mc, g, epi, s);
    default: return launch_tc_epi<32>(c, ma, mb, mc, g, epi, s);
  }
}

// fp32 CUDA-core GEMM whatever the precision mode: the timestep-conditioning tables built at weight load.
int gemm_f32(tsdp_ctx* c, const float* A, const float* W, const float* bias, int M, int N, int K, int epi, float* out,
             cudaStream_t s) {
  GemmArgs g{M, N, K, bias, out, N, c->status, nullptr, 0, nullptr, 1, 0, 1, 1, K, 0, LiveRows{nullptr, 0, 0}, nullptr, 0, 0, 0};
  dim3 grid((N + 63) / 64, (M + 63) / 64);
  if (epi == EPI_MISH) TSDP_LAUNCH(c, (gemm_simt_kernel<EPI_MISH>), grid, 256, 0, s, A, W, g);
  else if (epi == EPI_SILU) TSDP_LAUNCH(c, (gemm_simt_kernel<EPI_SILU>), grid, 256, 0, s, A, W, g);
  else TSDP_LAUNCH(c, (gemm_simt_kernel<EPI_F32>), grid, 256, 0, s, A, W, g);
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

// ------------------------------------------------------------------------------------------ nets
template <typename T>
int ln_launch(tsdp_ctx* c, const float* h, const float* g, const float* b, T* out, int M, int d, cudaStream_t s) {
  const int wpb = 8;
  const int grid = (M + wpb - 1) / wpb;
  prof_begin(c, s, 1, 0.0);
  switch (d / 128) {
    case 1: TSDP_LAUNCH(c, (ln_kernel<T, 1>), grid, wpb * 32, 0, s, h, g, b, out, M, live_desc(c, c->cfg.H)); break;
    case 2: TSDP_LAUNCH(c, (ln_kernel<T, 2>), grid, wpb * 32, 0, s, h, g, b, out, M, live_desc(c, c->cfg.H)); break;
    case 3: TSDP_LAUNCH(c, (ln_kernel<T, 3>), grid, wpb * 32, 0, s, h, g, b, out, M, live_desc(c, c->cfg.H)); break;
    case 4: TSDP_LAUNCH(c, (ln_kernel<T, 4>), grid, wpb * 32, 0, s, h, g, b, out, M, live_desc(c, c->cfg.H)); break;
    case 5: TSDP_LAUNCH(c, (ln_kernel<T, 5>), grid, wpb * 32, 0, s, h, g, b, out, M, live_desc(c, c->cfg.H)); break;
    case 6: TSDP_LAUNCH(c, (ln_kernel<T, 6>), grid, wpb * 32, 0, s, h, g, b, out, M, live_desc(c, c->cfg.H)); break;
    case 7: TSDP_LAUNCH(c, (ln_kernel<T, 7>), grid, wpb * 32, 0, s, h, g, b, out, M, live_desc(c, c->cfg.H)); break;
    default: TSDP_LAUNCH(c, (ln_kernel<T, 8>), grid, wpb * 32, 0, s, h, g, b, out, M, live_desc(c, c->cfg.H)); break;
  }
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

int head_launch(tsdp_ctx* c, const Net& n, const CandMap& cm, int M, cudaStream_t s) {
  const int wpb = 8;
  const int grid = (M + wpb - 1) / wpb;
  const int H = c->cfg.H, A = c->cfg.A;
#define HEAD_CASE(V) TSDP_LAUNCH(c, (head_kernel<V>), grid, wpb * 32, 0, s, c->h, n.lnf_g, n.lnf_b, n.W_outT, n.b_out, cm, M, H, A)
  prof_begin(c, s, 3, 0.0);
  switch (n.cfg.d / 128) {
    case 1: HEAD_CASE(1); break;
    case 2: HEAD_CASE(2); break;
    case 3: HEAD_CASE(3); break;
    case 4: HEAD_CASE(4); break;
    case 5: HEAD_CASE(5); break;
    case 6: HEAD_CASE(6); break;
    case 7: HEAD_CASE(7); break;
    default: HEAD_CASE(8); break;
  }
#undef HEAD_CASE
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

// Causal self-attention: tensor-core kernel for bf16 activations, the scalar kernel in check mode.
template <typename T>
int self_attn_launch(tsdp_ctx* c, const T* qkv, T* out, int n_cand, int H, int d, int heads, cudaStream_t s,
                     int causal = 1) {
  const int dh = d / heads;
  const LiveRows lv = live_desc(c, 1);
  prof_begin(c, s, 2, 0.0);
  if constexpr (std::is_same<T, __nv_bfloat16>::value) {
    const int QT = (H + 15) / 16;
    const int grid = (n_cand * heads * QT + SA_WARPS - 1) / SA_WARPS;
    if (H > 16 && (dh == 32 || dh == 64 || dh == 128)) {     // several query tiles share a head's K/V: stage them once
      const int g2 = n_cand * heads;
      if (dh == 32) TSDP_LAUNCH(c, (self_attn_staged_kernel<32>), g2, 128, 0, s, qkv, out, n_cand, H, d, heads, causal, lv);
      else if (dh == 64) TSDP_LAUNCH(c, (self_attn_staged_kernel<64>), g2, 128, 0, s, qkv, out, n_cand, H, d, heads, causal, lv);
      else TSDP_LAUNCH(c, (self_attn_staged_kernel<128>), g2, 128, 0, s, qkv, out, n_cand, H, d, heads, causal, lv);
    } else if (H <= 16 && (dh == 32 || dh == 64 || dh == 128)) {   // one 16-row tile: operands staged per warp
      const int tw = dh > 64 ? 2 : 4, g3 = (n_cand * heads + tw - 1) / tw;
      if (dh == 32) TSDP_LAUNCH(c, (self_attn_tile_kernel<32>), g3, tw * 32, 0, s, qkv, out, n_cand, H, d, heads, causal, lv);
      else if (dh == 64) TSDP_LAUNCH(c, (self_attn_tile_kernel<64>), g3, tw * 32, 0, s, qkv, out, n_cand, H, d, heads, causal, lv);
      else TSDP_LAUNCH(c, (self_attn_tile_kernel<128>), g3, tw * 32, 0, s, qkv, out, n_cand, H, d, heads, causal, lv);
    } else
    switch (dh) {
      case 32: TSDP_LAUNCH(c, (self_attn_mma_kernel<32>), grid, SA_WARPS * 32, 0, s, qkv, out, n_cand, H, d, heads, causal, lv); break;
      case 64: TSDP_LAUNCH(c, (self_attn_mma_kernel<64>), grid, SA_WARPS * 32, 0, s, qkv, out, n_cand, H, d, heads, causal, lv); break;
      case 96: TSDP_LAUNCH(c, (self_attn_mma_kernel<96>), grid, SA_WARPS * 32, 0, s, qkv, out, n_cand, H, d, heads, causal, lv); break;
      default: TSDP_LAUNCH(c, (self_attn_mma_kernel<128>), grid, SA_WARPS * 32, 0, s, qkv, out, n_cand, H, d, heads, causal, lv); break;
    }
  } else {
    const size_t per_warp = (size_t)(H * dh + 2 * H * (dh + 1)) * sizeof(float);
    int wpb = (int)((200 * 1024) / per_warp);      // the opt-in shared-memory limit set at init
    wpb = wpb > 4 ? 4 : (wpb < 1 ? 1 : wpb);
    const size_t smem = (size_t)wpb * per_warp;
    TSDP_LAUNCH(c, (self_attn_kernel<T>), (n_cand * heads + wpb - 1) / wpb, wpb * 32, smem, s, qkv, out, n_cand, H, d, heads, causal, lv);
  }
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

// Cross-attention to [time token | obs tokens]: register-resident keys/values when there are at most
// CA_MAXNK memory tokens and the head width is a power of two, the one-warp-per-row kernel otherwise.
template <typename T>
int cross_attn_launch(tsdp_ctx* c, const Net& n, const T* q2, T* out, const CandMap& cm, int n_cand, int layer,
                      cudaStream_t s) {
  const int H = c->cfg.H, d = n.cfg.d, heads = n.cfg.heads, L = n.cfg.layers, To = c->cfg.obs_tokens;
  const int dh = d / heads, M = n_cand * H;
  prof_begin(c, s, 2, 0.0);
  bool done = false;
  if constexpr (std::is_same<T, __nv_bfloat16>::value) {
    if (1 + To <= CA_MAXNK && (dh == 32 || dh == 64 || dh == 128)) {
      const long long threads = (long long)n_cand * heads * ((H + CA_ROWS - 1) / CA_ROWS) * (dh / 8);
      const int grid = (int)((threads + 255) / 256);
#define CA_CASE(DH) TSDP_LAUNCH(c, (cross_attn_group_kernel<DH>), grid, 256, 0, s, q2, out, n.kv_time, n.kv_obs, cm, n_cand, H, d, heads, To, layer, L, c->cfg.T)
      if (dh == 32) CA_CASE(32); else if (dh == 64) CA_CASE(64); else CA_CASE(128);
#undef CA_CASE
      done = true;
    }
  }
  if (!done)
    TSDP_LAUNCH(c, (cross_attn_kernel<T>), (M + 7) / 8, 256, 0, s, q2, out, n.kv_time, n.kv_obs, cm, M, H, d, heads, To, layer, L, c->cfg.T);
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

// Whether the QKV projection and the causal self-attention of this net run as one tensor-core kernel (EPI_ATTN).
bool fused_attn_ok(const tsdp_config_t& cfg, const tsdp_net_t& net) {
  return cfg.precision == 1 && net.arch == TSDP_ARCH_XFMR && cfg.H == 16 && net.heads > 0 && net.d / net.heads == 64 &&
         getenv("TSDP_NO_FUSED_ATTN") == nullptr;
}

// a [M, d] -> attention output [M, d]: QKV projection (head-major weights) with the 16-token causal self-attention in
// the GEMM's epilogue.  M is a multiple of 16 (whole candidates).
int gemm_qkv_attn(tsdp_ctx* c, const void* A, const XfmrLayer& w, int M, int d, void* out, cudaStream_t s) {
  const int N = 3 * d, K = d, BN = GEMM_ATTN_BN;
  GemmArgs g{M, N, K, w.bqkv_hm, out, d, c->status, nullptr, 0, nullptr, 1, 0, 1, 1, K, 0, LiveRows{nullptr, 0, 0}, nullptr, 0, 0, 1};
  if (c->live_n != nullptr && c->live_static > 0 && M % c->live_static == 0) g.live = LiveRows{c->live_n, M / c->live_static, 0};
  CUtensorMap ma, mb;
  int r;
  if ((r = get_map(c, A, 2, M, K, K, GEMM_BK, GEMM_BM, &ma)) != TSDP_OK) return r;
  const long long ptiles = (long long)((M + 255) / 256) * (N / BN);
  const bool pair = c->pair_mode == 2 && c->pair_clusters_attn >= 1;      // K = d <= 1024 here: the single-CTA form is as fast
  if ((r = get_map(c, w.Wqkv_hm, 2, N, K, K, GEMM_BK, pair ? BN / 2 : BN, &mb)) != TSDP_OK) return r;
  prof_begin(c, s, c->prof_gemm_cat, 2.0 * gemm_rows_known(c, g) * N * K);
  if (pair) {
    const int pairs = ptiles < c->pair_clusters_attn ? (int)ptiles : c->pair_clusters_attn;
    launch_kernel_cluster(c, gemm_tcgen05_kernel<GEMM_ATTN_BN, EPI_ATTN, 2>, dim3(2 * pairs), dim3(GEMM_THREADS),
                          (size_t)gemm_smem_bytes_cg(BN, 2), s, 2, ma, mb, ma, g);
  } else {
    const int tiles = ((M + GEMM_BM - 1) / GEMM_BM) * (N / BN);
    const int grid = tiles < c->num_sms ? tiles : c->num_sms;
    TSDP_LAUNCH(c, (gemm_tcgen05_kernel<GEMM_ATTN_BN, EPI_ATTN>), grid, GEMM_THREADS, gemm_smem_bytes(BN), s, ma, mb, ma, g);
  }
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

int gemm_qkv_attn_raw(tsdp_ctx* c, const void* A, const void* W_hm, const float* b_hm, int M, int d, void* out, cudaStream_t s) {
  XfmrLayer w{};
  w.Wqkv_hm = const_cast<void*>(W_hm);
  w.bqkv_hm = const_cast<float*>(b_hm);
  return gemm_qkv_attn(c, A, w, M, d, out, s);
}

// Whether the cross-attention sub-block of this net runs folded into its memory tokens (xattn_fold.cuh).
bool xfold_ok(const tsdp_config_t& cfg, const tsdp_net_t& net) {
  if (cfg.precision != 1 || net.arch != TSDP_ARCH_XFMR || getenv("TSDP_NO_FOLD") != nullptr) return false;
  const int NK = 1 + cfg.obs_tokens, d = net.d, heads = net.heads;
  if (heads < 2 || heads > 16 || heads % 2 || d % heads) return false;      // one (row, head) of the softmax per thread
  const int dh = d / heads;
  return cfg.H <= 16 && NK <= XF_MAXNK && NK * heads <= XF_MAXN && (d == 128 || d == 256 || d == 512) &&
         dh % 8 == 0 && dh <= 128 && xfold_build_smem(d, dh) <= 200 * 1024;
}

// Fold tables of `rows` memory tokens (keys / values kv, row pitch L*2d) of net n.
int xfold_build(tsdp_ctx* c, Net& n, const float* kv, int rows, __nv_bfloat16* kq, __nv_bfloat16* ut, float* cc, cudaStream_t s) {
  const int d = n.cfg.d, heads = n.cfg.heads, L = n.cfg.layers;
  int splits = (2 * c->num_sms + L * heads - 1) / (L * heads);
  const int groups = (rows + XF_RB - 1) / XF_RB;
  if (splits > groups) splits = groups;
  if (splits < 1) splits = 1;
  prof_begin(c, s, 3, 0.0);
  xfold_build_kernel<<<dim3(L * heads, splits), 256, xfold_build_smem(d, d / heads), s>>>(kv, (long long)L * 2 * d, rows, n.fold_lw, L,
                                                                                          d, heads, kq, ut, cc);
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

int xattn_fold_launch(tsdp_ctx* c, const Net& n, const XfmrLayer& w, const __nv_bfloat16* delta, __nv_bfloat16* ln3_out,
                      const CandMap& cm, int n_cand, int layer, cudaStream_t s) {
  const int H = c->cfg.H, d = n.cfg.d, heads = n.cfg.heads, L = n.cfg.layers, To = c->cfg.obs_tokens;
  const XfoldTables tb{n.fold_kq_time, n.fold_ut_time, n.fold_c_time, n.fold_kq_obs, n.fold_ut_obs, n.fold_c_obs};
  prof_begin(c, s, 2, 0.0);
#define XF_CASE(DD) TSDP_LAUNCH(c, (xattn_fold_kernel<DD>), n_cand, XF_THREADS, xf_smem_bytes(DD, (1 + To) * heads), s, c->h, delta, tb, w.bo2, w.ln3_g, w.ln3_b, ln3_out, cm, H, heads, To, layer, L, c->cfg.T)
  switch (d) {
    case 128: XF_CASE(128); break;
    case 256: XF_CASE(256); break;
    default: XF_CASE(512); break;
  }
#undef XF_CASE
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

template <typename T>
int xfmr_forward_t(tsdp_ctx* c, Net& n, const CandMap& cm, int n_cand, cudaStream_t s) {
  const int H = c->cfg.H, A = c->cfg.A, d = n.cfg.d, heads = n.cfg.heads, L = n.cfg.layers;
  const int M = n_cand * H;
  const int dh = d / heads;
  T* a = reinterpret_cast<T*>(c->a);
  T* qkv = reinterpret_cast<T*>(c->qkv);
  T* q2 = reinterpret_cast<T*>(c->q2);
  T* f = reinterpret_cast<T*>(c->f);
  int r;
  if (!c->xf_skip_embed) {   // token embedding and the first block's LayerNorm
    const int wpb = 8, grid = (M + wpb - 1) / wpb;
    const XfmrLayer& w0 = n.L[0];
    prof_begin(c, s, 3, 0.0);
#define EL_CASE(V) TSDP_LAUNCH(c, (embed_ln_kernel<T, V>), grid, wpb * 32, 0, s, cm, n.W_in, n.b_in, n.pos, c->h, w0.ln1_g, w0.ln1_b, a, M, H, A)
    switch (d / 128) {
      case 1: EL_CASE(1); break; case 2: EL_CASE(2); break; case 3: EL_CASE(3); break; case 4: EL_CASE(4); break;
      case 5: EL_CASE(5); break; case 6: EL_CASE(6); break; case 7: EL_CASE(7); break; default: EL_CASE(8); break;
    }
#undef EL_CASE
    prof_end(c, s);
    c->launches_per_round_tmp++;
    CU_TRY(c, cudaGetLastError());
  }
  const int out_epi = (c->cfg.precision == 0) ? EPI_F32 : EPI_STORE;
  for (int l = 0; l < L; ++l) {
    const XfmrLayer& w = n.L[l];
    if (l > 0 && (r = ln_launch<T>(c, c->h, w.ln1_g, w.ln1_b, a, M, d, s))) return r;
    if (w.Wqkv_hm != nullptr && std::is_same<T, __nv_bfloat16>::value) {
      // QKV projection and self-attention in one kernel: q, k, v never reach memory.  Its output goes to q2 (the
      // kernel reads `a` while it writes) and is then the operand of the attention projection.
      if ((r = gemm_qkv_attn(c, a, w, M, d, q2, s))) return r;
      std::swap(a, q2);
    } else {
      if ((r = gemm(c, a, w.Wqkv, w.bqkv, M, 3 * d, d, out_epi, qkv, 3 * d, s))) return r;
      if ((r = self_attn_launch<T>(c, qkv, a, n_cand, H, d, heads, s))) return r;
    }
    if (n.fold) {
      // the attention projection leaves as bf16; the fold kernel adds it to the stream, does the cross-attention
      // sub-block and the LayerNorm in front of the MLP
      if ((r = gemm(c, a, w.Wo, w.bo, M, d, d, EPI_STORE, q2, d, s))) return r;
      if ((r = xattn_fold_launch(c, n, w, reinterpret_cast<const __nv_bfloat16*>(q2), reinterpret_cast<__nv_bfloat16*>(a), cm, n_cand, l, s)))
        return r;
    } else {
      if ((r = gemm(c, a, w.Wo, w.bo, M, d, d, EPI_RESID, c->h, d, s))) return r;
      if ((r = ln_launch<T>(c, c->h, w.ln2_g, w.ln2_b, a, M, d, s))) return r;
      if ((r = gemm(c, a, w.Wq2, w.bq2, M, d, d, out_epi, q2, d, s))) return r;
      if ((r = cross_attn_launch<T>(c, n, q2, a, cm, n_cand, l, s))) return r;
      if ((r = gemm(c, a, w.Wo2, w.bo2, M, d, d, EPI_RESID, c->h, d, s))) return r;
      if ((r = ln_launch<T>(c, c->h, w.ln3_g, w.ln3_b, a, M, d, s))) return r;
    }
    if ((r = gemm(c, a, w.W1, w.b1, M, 4 * d, d, EPI_GELU, f, 4 * d, s))) return r;
    if ((r = gemm(c, f, w.W2, w.b2, M, d, 4 * d, EPI_RESID, c->h, d, s))) return r;
  }
  if (c->xf_skip_head) return TSDP_OK;
  return head_launch(c, n, cm, M, s);
}

// Head of the drafter, the draft step and the next step's embedding + LayerNorm in one launch (draft_tail.cuh).
template <typename T>
int draft_tail_launch(tsdp_ctx* c, Net& n, int B, int k, int K, bool embed_next, cudaStream_t s, const int* order,
                      const int* n_live) {
  const int H = c->cfg.H, A = c->cfg.A, D = c->D, M = B * H, d = n.cfg.d;
  const long long xs_b = (long long)(c->cfg.max_K + 1) * D, ms_b = (long long)(c->cfg.max_K > 0 ? c->cfg.max_K : 1) * D;
  const int wpb = 8, grid = (M + wpb - 1) / wpb;
  const XfmrLayer& w0 = n.L[0];
  T* a = reinterpret_cast<T*>(c->a);
  prof_begin(c, s, 4, 0.0);
#define DT_CASE(V) TSDP_LAUNCH(c, (draft_tail_kernel<T, V>), grid, wpb * 32, 0, s, c->h, n.lnf_g, n.lnf_b, n.W_outT, n.b_out, c->S, c->xt, xs_b, \
                               c->muhat, ms_b, c->eps_d, c->t, k, K, c->cfg.T, c->seed, c->sched_on ? c->envp : nullptr, c->item, n.W_in, n.b_in,   \
                               n.pos, w0.ln1_g, w0.ln1_b, a, embed_next ? 1 : 0, M, H, A, order, n_live)
  switch (d / 128) {
    case 1: DT_CASE(1); break; case 2: DT_CASE(2); break; case 3: DT_CASE(3); break; case 4: DT_CASE(4); break;
    case 5: DT_CASE(5); break; case 6: DT_CASE(6); break; case 7: DT_CASE(7); break; default: DT_CASE(8); break;
  }
#undef DT_CASE
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

// Observation tokens -> their cross-attention keys/values for every block (once per chunk).
template <typename T>
int xfmr_prepare_obs_t(tsdp_ctx* c, Net& n, int B, cudaStream_t s) {
  const int To = c->cfg.obs_tokens, d = n.cfg.d, L = n.cfg.layers;
  if (To == 0) return TSDP_OK;
  T* mt = reinterpret_cast<T*>(c->memtok);
  prof_begin(c, s, 3, 0.0);
  TSDP_LAUNCH(c, (memtok_kernel<T>), B * To, d < 256 ? d : 256, 0, s, c->obs, c->cfg.obs_dim, n.W_obs, n.b_obs, n.cpos, To, 1, mt, d);
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  int r = gemm(c, mt, n.Wkv_all, n.bkv_all, B * To, L * 2 * d, d, EPI_F32, n.kv_obs, L * 2 * d, s);
  if (r || !n.fold) return r;
  return xfold_build(c, n, n.kv_obs, B * To, n.fold_kq_obs, n.fold_ut_obs, n.fold_c_obs, s);
}

// ------------------------------------------------------------------------------------------ DiT
template <typename T>
int ln_mod_launch(tsdp_ctx* c, const Net& n, int off_shift, int off_scale, const CandMap& cm, T* out, int M, cudaStream_t s) {
  const int wpb = 8, grid = (M + wpb - 1) / wpb, H = c->cfg.H, Ts = c->cfg.T;
  prof_begin(c, s, 1, 0.0);
#define LNM_CASE(V) TSDP_LAUNCH(c, (ln_mod_kernel<T, V>), grid, wpb * 32, 0, s, c->h, n.mod, n.mod_ld, off_shift, off_scale, cm, H, Ts, out, M)
  switch (n.cfg.d / 128) {
    case 1: LNM_CASE(1); break; case 2: LNM_CASE(2); break; case 3: LNM_CASE(3); break; case 4: LNM_CASE(4); break;
    case 5: LNM_CASE(5); break; case 6: LNM_CASE(6); break; case 7: LNM_CASE(7); break; default: LNM_CASE(8); break;
  }
#undef LNM_CASE
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

// Cross-attention of every candidate's tokens to the context tokens of its request.
template <typename T>
int cross_attn_ctx_launch(tsdp_ctx* c, const Net& n, const T* q2, T* out, const CandMap& cm, int n_cand, int layer,
                          cudaStream_t s) {
  const int H = c->cfg.H, d = n.cfg.d, heads = n.cfg.heads, L = n.cfg.layers, Tc = c->cfg.obs_tokens;
  const int dh = d / heads, M = n_cand * H;
  const long long ld_kv = (long long)L * 2 * d;
  const T* kv = reinterpret_cast<const T*>(n.kv_obs);
  bool done = false;
  if constexpr (std::is_same<T, __nv_bfloat16>::value) {
    // 64-wide heads and groups of at least two 128-row tiles (the verification forward: all candidates of a slot share
    // the keys / values a CTA fetched): both products on the 5th-generation tensor cores (ctx_attn_tcgen05.cuh).
    // Measured on the VLA-scale workload: a quarter less attention time than the mma.sync kernel there (55 vs 75 ms of
    // the step), but no faster for the drafter's single 50-row group per CTA, where fetching and re-laying-out K / V
    // dominates; tc_attn = 2 forces it.
    if (c->tc_attn && (cm.C * H >= 256 || c->tc_attn == 2) && dh == 64 && Tc % 32 == 0 && Tc <= 256 && n_cand % cm.C == 0 && d % 8 == 0) {
      const int slots = n_cand / cm.C, rows = cm.C * H;
      CUtensorMap mq, mkv;
      int r;
      if ((r = get_map(c, q2, 2, M, d, d, 64, 128, &mq)) != TSDP_OK) return r;
      if ((r = get_map(c, kv, 2, (int)(c->items_cap * (size_t)Tc), L * 2 * d, L * 2 * d, 64, Tc, &mkv)) != TSDP_OK) return r;
      prof_begin(c, s, 2, 0.0);
      TSDP_LAUNCH(c, (cross_attn_ctx_tc_kernel), slots * heads, CXT_THREADS, CXT_SMEM_BYTES, s, mq, mkv, reinterpret_cast<__nv_bfloat16*>(out),
                  layer * 2 * d, cm, rows, d, heads, Tc, c->live_slot_start, H, c->status);
      prof_end(c, s);
      c->launches_per_round_tmp++;
      CU_TRY(c, cudaGetLastError());
      return TSDP_OK;
    }
  }
  prof_begin(c, s, 2, 0.0);
  if constexpr (std::is_same<T, __nv_bfloat16>::value) {
    if (Tc % 16 == 0 && (dh == 32 || dh == 64 || dh == 128) && n_cand % cm.C == 0) {
      const int slots = n_cand / cm.C, rows = cm.C * H;
#define CX_CASE(DH) TSDP_LAUNCH(c, (cross_attn_ctx_mma_kernel<DH>), slots * heads, CX_WARPS * 32, cx_smem_bytes<DH>(Tc), s, q2, out, kv, ld_kv, layer * 2 * d, cm, rows, d, heads, Tc, c->live_slot_start, H)
      if (dh == 32) CX_CASE(32); else if (dh == 64) CX_CASE(64); else CX_CASE(128);
#undef CX_CASE
      done = true;
    }
  }
  if (!done) {
    const int wpb = 4;
    TSDP_LAUNCH(c, (cross_attn_ctx_simt_kernel<T>), (M + wpb - 1) / wpb, wpb * 32, (size_t)wpb * Tc * sizeof(float), s, q2, out,
                kv, ld_kv, layer * 2 * d, cm, M, H, d, heads, Tc);
  }
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

template <typename T>
int dit_forward_t(tsdp_ctx* c, Net& n, const CandMap& cm, int n_cand, cudaStream_t s) {
  const int H = c->cfg.H, A = c->cfg.A, d = n.cfg.d, heads = n.cfg.heads, L = n.cfg.layers;
  const int M = n_cand * H;
  T* a = reinterpret_cast<T*>(c->a);
  T* qkv = reinterpret_cast<T*>(c->qkv);
  T* q2 = reinterpret_cast<T*>(c->q2);
  T* f = reinterpret_cast<T*>(c->f);
  int r;
  prof_begin(c, s, 3, 0.0);
  TSDP_LAUNCH(c, (embed_kernel), M, d < 256 ? d : 256, 0, s, cm, n.W_in, n.b_in, n.pos, c->h, H, A, d);
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  const int out_epi = (c->cfg.precision == 0) ? EPI_F32 : EPI_STORE;
  for (int l = 0; l < L; ++l) {
    const XfmrLayer& w = n.L[l];
    const int base = l * 6 * d;        // (shift1, scale1, gate1, shift2, scale2, gate2) of this block in a row of mod
    GateSpec g1{n.mod + base + 2 * d, n.mod_ld, &cm, H, c->cfg.T}, g2{n.mod + base + 5 * d, n.mod_ld, &cm, H, c->cfg.T};
    if ((r = ln_mod_launch<T>(c, n, base, base + d, cm, a, M, s))) return r;
    if ((r = gemm(c, a, w.Wqkv, w.bqkv, M, 3 * d, d, out_epi, qkv, 3 * d, s))) return r;
    if ((r = self_attn_launch<T>(c, qkv, a, n_cand, H, d, heads, s, 0))) return r;
    if ((r = gemm(c, a, w.Wo, w.bo, M, d, d, EPI_GATE, c->h, d, s, &g1))) return r;
    if ((r = ln_launch<T>(c, c->h, w.ln2_g, w.ln2_b, a, M, d, s))) return r;
    if ((r = gemm(c, a, w.Wq2, w.bq2, M, d, d, out_epi, q2, d, s))) return r;
    if ((r = cross_attn_ctx_launch<T>(c, n, q2, a, cm, n_cand, l, s))) return r;
    if ((r = gemm(c, a, w.Wo2, w.bo2, M, d, d, EPI_RESID, c->h, d, s))) return r;
    if ((r = ln_mod_launch<T>(c, n, base + 3 * d, base + 4 * d, cm, a, M, s))) return r;
    if ((r = gemm(c, a, w.W1, w.b1, M, 4 * d, d, EPI_GELU, f, 4 * d, s))) return r;
    if ((r = gemm(c, f, w.W2, w.b2, M, d, 4 * d, EPI_GATE, c->h, d, s, &g2))) return r;
  }
  const int wpb = 8, grid = (M + wpb - 1) / wpb, offf = L * 6 * d;
  prof_begin(c, s, 3, 0.0);
#define HM_CASE(V) TSDP_LAUNCH(c, (head_mod_kernel<V>), grid, wpb * 32, 0, s, c->h, n.mod, n.mod_ld, offf, offf + d, n.W_outT, n.b_out, cm, M, H, A, c->cfg.T)
  switch (d / 128) {
    case 1: HM_CASE(1); break; case 2: HM_CASE(2); break; case 3: HM_CASE(3); break; case 4: HM_CASE(4); break;
    case 5: HM_CASE(5); break; case 6: HM_CASE(6); break; case 7: HM_CASE(7); break; default: HM_CASE(8); break;
  }
#undef HM_CASE
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

// Context tokens -> their cross-attention keys/values for every block (once per chunk), in the
// activation type (they are tensor-core operands of the attention kernel).
template <typename T>
int dit_prepare_ctx_t(tsdp_ctx* c, Net& n, int B, cudaStream_t s) {
  const int Tc = c->cfg.obs_tokens, d = n.cfg.d, L = n.cfg.layers;
  T* mt = reinterpret_cast<T*>(c->memtok);
  prof_begin(c, s, 3, 0.0);
  TSDP_LAUNCH(c, (memtok_kernel<T>), B * Tc, d < 256 ? d : 256, 0, s, c->obs, c->cfg.obs_dim, n.W_obs, n.b_obs, n.cpos, Tc, 0, mt, d);
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return gemm(c, mt, n.Wkv_all, n.bkv_all, B * Tc, L * 2 * d, d, c->cfg.precision == 0 ? EPI_F32 : EPI_STORE, n.kv_obs,
              L * 2 * d, s);
}

// ------------------------------------------------------------------------------------------ conv UNet
template <typename T>
int unet_gn(tsdp_ctx* c, Net& n, const CandMap& cm, int n_cand, const float* gam, const float* bet, int foff, const T* res_t,
            int res_pitch, const float* res_f, T* dst, int dst_pitch, int coff, int L, int C, cudaStream_t s, int n_split = 1,
            long long split_stride = 0) {
  prof_begin(c, s, 1, 0.0);
  TSDP_LAUNCH(c, (gn_mish_kernel<T>), n_cand * n.cfg.heads, 256, 0, s, n.uw.Y, gam, bet, n.cfg.heads,
              foff >= 0 ? n.film_time : nullptr, n.film_obs, n.F, foff >= 0 ? foff : 0, cm, c->cfg.T, res_t, res_pitch, res_f, dst,
              dst_pitch, coff, L, C, n_split, split_stride);
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

// One FiLM residual block: xin [n, L+4, cin] -> dst[n, L+4, coff .. coff+cout) of a tensor of pitch dst_pitch.
template <typename T>
int unet_resblock(tsdp_ctx* c, Net& n, const Net::UBlock& b, const CandMap& cm, int n_cand, const T* xin, T* tmp, T* dst,
                  int dst_pitch, int coff, int L, cudaStream_t s) {
  const int rows = n_cand * (L + 4);
  int r;
  const long long ystr = (long long)rows * b.cout;      // distance of the partial-sum buffers of a split reduction
  const int s1 = conv_ksplit(c, rows - 4, b.cout, 5 * b.cin, n.uw.Y_cap), s2 = conv_ksplit(c, rows - 4, b.cout, 5 * b.cout, n.uw.Y_cap);
  const bool fork = b.Wr != nullptr && c->aux_on && !c->prof_on;      // (per-launch timing keeps one stream)
  if (fork) {      // the residual projection only needs xin: beside the two convolutions, on the second stream
    CU_TRY(c, cudaEventRecord(c->ev_aux_fork, s));
    CU_TRY(c, cudaStreamWaitEvent(c->aux_stream, c->ev_aux_fork, 0));
    if ((r = gemm(c, xin, b.Wr, b.br, rows, b.cout, b.cin, EPI_F32, n.uw.R, b.cout, c->aux_stream))) return r;
    CU_TRY(c, cudaEventRecord(c->ev_aux_join, c->aux_stream));
  }
  if ((r = gemm(c, xin, b.W1, b.b1, rows - 4, b.cout, 5 * b.cin, EPI_F32, n.uw.Y, b.cout, s, nullptr, b.cin, s1, ystr))) return r;
  if ((r = unet_gn<T>(c, n, cm, n_cand, b.g1, b.be1, b.foff, nullptr, 0, nullptr, tmp, b.cout, 0, L, b.cout, s, s1, ystr))) return r;
  if ((r = gemm(c, tmp, b.W2, b.b2, rows - 4, b.cout, 5 * b.cout, EPI_F32, n.uw.Y, b.cout, s, nullptr, b.cout, s2, ystr))) return r;
  if (b.Wr) {
    if (fork) CU_TRY(c, cudaStreamWaitEvent(s, c->ev_aux_join, 0));
    else if ((r = gemm(c, xin, b.Wr, b.br, rows, b.cout, b.cin, EPI_F32, n.uw.R, b.cout, s))) return r;
    return unet_gn<T>(c, n, cm, n_cand, b.g2, b.be2, -1, nullptr, 0, n.uw.R, dst, dst_pitch, coff, L, b.cout, s, s2, ystr);
  }
  return unet_gn<T>(c, n, cm, n_cand, b.g2, b.be2, -1, xin, b.cin, nullptr, dst, dst_pitch, coff, L, b.cout, s, s2, ystr);
}

template <typename T>
int unet_forward_t(tsdp_ctx* c, Net& n, const CandMap& cm, int n_cand, cudaStream_t s) {
  const int H = c->cfg.H, A = c->cfg.A, ch = n.cfg.d, LV = n.cfg.layers, last = LV - 1;
  auto P = [](void* p) { return reinterpret_cast<T*>(p); };
  int r, bi = 0;
  prof_begin(c, s, 3, 0.0);
  TSDP_LAUNCH(c, (unet_embed_kernel<T>), n_cand * H, ch < 256 ? ch : 256, 0, s, cm, n.W_in, n.b_in, P(n.uw.X0), H, A, ch);
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  const T* x = P(n.uw.X0);
  for (int lv = 0; lv < LV; ++lv) {
    const int L = H >> lv, C = ch << lv;
    if ((r = unet_resblock<T>(c, n, n.ub[bi++], cm, n_cand, x, P(n.uw.TMP[lv]), P(n.uw.D[lv]), C, 0, L, s))) return r;
    if (lv < last) {
      const int Cup = ch << (lv + 1), Ccat = Cup + C;
      if ((r = unet_resblock<T>(c, n, n.ub[bi++], cm, n_cand, P(n.uw.D[lv]), P(n.uw.TMP[lv]), P(n.uw.CAT[lv]), Ccat, Cup, L, s))) return r;
      const long long tot = (long long)n_cand * (L / 2) * C;
      prof_begin(c, s, 3, 0.0);
      TSDP_LAUNCH(c, (unet_pool_kernel<T>), (unsigned)((tot + 255) / 256), 256, 0, s, P(n.uw.CAT[lv]), Ccat, Cup, P(n.uw.P[lv]),
                  n_cand, L / 2, C, live_desc(c, 1));
      prof_end(c, s);
      c->launches_per_round_tmp++;
      CU_TRY(c, cudaGetLastError());
      x = P(n.uw.P[lv]);
    } else {
      if ((r = unet_resblock<T>(c, n, n.ub[bi++], cm, n_cand, P(n.uw.D[lv]), P(n.uw.TMP[lv]), P(n.uw.E), C, 0, L, s))) return r;
    }
  }
  {
    const int L = H >> last, C = ch << last;
    if ((r = unet_resblock<T>(c, n, n.ub[bi++], cm, n_cand, P(n.uw.E), P(n.uw.TMP[last]), P(n.uw.M1), C, 0, L, s))) return r;
    if ((r = unet_resblock<T>(c, n, n.ub[bi++], cm, n_cand, P(n.uw.M1), P(n.uw.TMP[last]), P(n.uw.M2), C, 0, L, s))) return r;
  }
  const T* cur = P(n.uw.M2);
  for (int lv = last - 1; lv >= 0; --lv) {
    const int L = H >> lv, C = ch << lv, Cup = ch << (lv + 1), Ccat = Cup + C;
    const long long tot = (long long)n_cand * L * Cup;
    prof_begin(c, s, 3, 0.0);
    TSDP_LAUNCH(c, (unet_upsample_kernel<T>), (unsigned)((tot + 255) / 256), 256, 0, s, cur, P(n.uw.CAT[lv]), Ccat, n_cand, L, Cup, live_desc(c, 1));
    prof_end(c, s);
    c->launches_per_round_tmp++;
    CU_TRY(c, cudaGetLastError());
    if ((r = unet_resblock<T>(c, n, n.ub[bi++], cm, n_cand, P(n.uw.CAT[lv]), P(n.uw.TMP[lv]), P(n.uw.U1[lv]), C, 0, L, s))) return r;
    if ((r = unet_resblock<T>(c, n, n.ub[bi++], cm, n_cand, P(n.uw.U1[lv]), P(n.uw.TMP[lv]), P(n.uw.U2[lv]), C, 0, L, s))) return r;
    cur = P(n.uw.U2[lv]);
  }
  const int rows = n_cand * (H + 4);
  const long long ystr = (long long)rows * ch;
  const int sh = conv_ksplit(c, rows - 4, ch, 5 * ch, n.uw.Y_cap);
  if ((r = gemm(c, cur, n.Wh, n.bh, rows - 4, ch, 5 * ch, EPI_F32, n.uw.Y, ch, s, nullptr, ch, sh, ystr))) return r;
  if ((r = unet_gn<T>(c, n, cm, n_cand, n.gh, n.beh, -1, nullptr, 0, nullptr, P(n.uw.HB), ch, 0, H, ch, s, sh, ystr))) return r;
  prof_begin(c, s, 3, 0.0);
  TSDP_LAUNCH(c, (unet_head_kernel<T>), (n_cand * H + 7) / 8, 256, 0, s, P(n.uw.HB), n.W_outT, n.b_out, cm, n_cand * H, H, A, ch);
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

// FiLM contribution of every request's observation: film_obs = Mish(obs_flat) Wf_obs (once per chunk).
int unet_prepare_obs(tsdp_ctx* c, Net& n, int N, cudaStream_t s) {
  const int dobs = c->cfg.obs_tokens * c->cfg.obs_dim;
  if (dobs == 0) return TSDP_OK;
  const long long tot = (long long)N * dobs;
  TSDP_LAUNCH(c, (mish_kernel), (unsigned)((tot + 255) / 256), 256, 0, s, c->obs, n.obs_m, tot);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  c->launches_per_round_tmp++;
  return gemm_f32(c, n.obs_m, n.WfT_obs, nullptr, N, n.F, dobs, EPI_F32, n.film_obs, s);
}

int prepare_obs(tsdp_ctx* c, Net& n, int B, cudaStream_t s) {
  if (n.cfg.arch == TSDP_ARCH_UNET) return unet_prepare_obs(c, n, B, s);
  if (n.cfg.arch == TSDP_ARCH_DIT)
    return c->cfg.precision == 0 ? dit_prepare_ctx_t<float>(c, n, B, s) : dit_prepare_ctx_t<__nv_bfloat16>(c, n, B, s);
  if (n.cfg.arch != TSDP_ARCH_XFMR) return TSDP_OK;
  return c->cfg.precision == 0 ? xfmr_prepare_obs_t<float>(c, n, B, s) : xfmr_prepare_obs_t<__nv_bfloat16>(c, n, B, s);
}

int forward_arch(tsdp_ctx* c, Net& n, const CandMap& cm, int n_cand, cudaStream_t s);

// One network forward over the candidates of `cm`.  With a compacted list the launches are still sized for n_cand
// (the dense count, so that a captured graph stays valid) and every kernel reads the live count from the device.
int forward(tsdp_ctx* c, Net& n, const CandMap& cm, int n_cand, cudaStream_t s, const int* slot_start = nullptr) {
  if (n_cand <= 0) return TSDP_OK;
  c->live_n = cm.n_live;
  c->live_static = n_cand;
  c->live_slot_start = cm.list ? slot_start : nullptr;
  const int r = forward_arch(c, n, cm, n_cand, s);
  c->live_n = nullptr; c->live_static = 0; c->live_slot_start = nullptr;
  return r;
}

int forward_arch(tsdp_ctx* c, Net& n, const CandMap& cm, int n_cand, cudaStream_t s) {
  const int D = c->D;
  switch (n.cfg.arch) {
    case TSDP_ARCH_GAUSS: {
      const long long tot = (long long)n_cand * D;
      prof_begin(c, s, 5, 0.0);
      TSDP_LAUNCH(c, (gauss_forward_kernel), (unsigned)((tot + 255) / 256), 256, 0, s, c->S, n.m0, n.s0, cm, n_cand, D);
      prof_end(c, s);
      c->launches_per_round_tmp++;
      CU_TRY(c, cudaGetLastError());
      return TSDP_OK;
    }
    case TSDP_ARCH_MLP: {
      int maxw = 0;
      for (int l = 0; l <= n.mlp.n_lin; ++l) maxw = n.mlp.dims[l] > maxw ? n.mlp.dims[l] : maxw;
      prof_begin(c, s, 5, 0.0);
      TSDP_LAUNCH(c, (mlp_forward_kernel), n_cand, 256, 2 * maxw * sizeof(float), s, n.mlp, cm, c->obs, c->cfg.obs_tokens * c->cfg.obs_dim,
                                                                        D, c->cfg.T);
      prof_end(c, s);
      c->launches_per_round_tmp++;
      CU_TRY(c, cudaGetLastError());
      return TSDP_OK;
    }
    case TSDP_ARCH_XFMR:
      return c->cfg.precision == 0 ? xfmr_forward_t<float>(c, n, cm, n_cand, s)
                                   : xfmr_forward_t<__nv_bfloat16>(c, n, cm, n_cand, s);
    case TSDP_ARCH_DIT:
      return c->cfg.precision == 0 ? dit_forward_t<float>(c, n, cm, n_cand, s)
                                   : dit_forward_t<__nv_bfloat16>(c, n, cm, n_cand, s);
    case TSDP_ARCH_UNET:
      return c->cfg.precision == 0 ? unet_forward_t<float>(c, n, cm, n_cand, s)
                                   : unet_forward_t<__nv_bfloat16>(c, n, cm, n_cand, s);
  }
  return TSDP_ERR_UNSUPPORTED;
}

// ------------------------------------------------------------------------------------------ drafter
// Whether the persistent cluster kernel can run this context's drafter at all (shapes, shared memory).
bool cluster_drafter_fits(const tsdp_config_t& cfg, const tsdp_net_t& n, int* smem_bytes, bool* resident) {
  if (cfg.precision != 1 || n.arch != TSDP_ARCH_XFMR || (n.d != 128 && n.d != 256) || n.layers > DC_MAX_LAYERS ||
      cfg.H > DC_ROWS || 1 + cfg.obs_tokens > DC_MAX_NK || cfg.H * cfg.A > 256 || (n.d / n.heads) % 4 != 0)
    return false;
  // weight slices resident in shared memory if they fit beside the activations, otherwise read through the L2
  for (int res = 1; res >= 0; --res) {
    const DcSmem pl = dc_smem_plan(n.d, n.layers, cfg.A, res != 0);
    if (pl.total <= 227 * 1024) { *smem_bytes = pl.total; *resident = res != 0; return true; }
  }
  return false;
}

bool use_cluster_drafter(const tsdp_ctx* c, int B) {
  if (!c->dc_ok || c->cfg.drafter == 1) return false;
  if (c->cfg.drafter == 2) return true;
  // Beyond a few waves of clusters the batched tensor-core path wins: measured about 29 us per draft step and wave
  // with resident weights (PushT drafter) and 70-130 us with L2-streamed ones, against 100-175 us per step for the
  // layer-by-layer path whatever the batch.
  return B <= (c->dc_resident ? 3 : 1) * c->dc_max_clusters;
}

bool use_cluster_verifier(const tsdp_ctx* c, int B, int K) {
  if (!c->cv_ok || c->cfg.verifier == 1) return false;
  if (c->cfg.verifier == 2) return true;
  return B * (K + 1) <= c->cv_max_clusters;     // every candidate gets its own cluster in one wave
}

// mode 0: K-step draft rollout with the drafter; mode 1: verification forward of the base model on K+1 candidates.
int launch_cluster_forward(tsdp_ctx* c, int which, int mode, int B, int K, cudaStream_t s) {
  const Net& n = c->net[which];
  DcParams P{};
  for (int l = 0; l < n.cfg.layers; ++l) {
    const XfmrLayer& w = n.L[l];
    DcLayer& o = P.L[l];
    o.Wqkv = (const __nv_bfloat16*)w.Wqkv; o.Wo = (const __nv_bfloat16*)w.Wo; o.Wq2 = (const __nv_bfloat16*)w.Wq2;
    o.Wo2 = (const __nv_bfloat16*)w.Wo2; o.W1 = (const __nv_bfloat16*)w.W1; o.W2 = (const __nv_bfloat16*)w.W2;
    o.bqkv = w.bqkv; o.bo = w.bo; o.bq2 = w.bq2; o.bo2 = w.bo2; o.b1 = w.b1; o.b2 = w.b2;
    o.ln1_g = w.ln1_g; o.ln1_b = w.ln1_b; o.ln2_g = w.ln2_g; o.ln2_b = w.ln2_b; o.ln3_g = w.ln3_g; o.ln3_b = w.ln3_b;
  }
  P.layers = n.cfg.layers; P.heads = n.cfg.heads; P.H = c->cfg.H; P.A = c->cfg.A; P.To = c->cfg.obs_tokens; P.T = c->cfg.T;
  P.W_in = n.W_in; P.b_in = n.b_in; P.pos = n.pos;
  P.lnf_g = n.lnf_g; P.lnf_b = n.lnf_b; P.W_outT = n.W_outT; P.b_out = n.b_out;
  P.kv_time = n.kv_time; P.kv_obs = n.kv_obs;
  P.fold = (n.fold && (1 + c->cfg.obs_tokens) * n.cfg.heads <= 16) ? 1 : 0;     // the cluster kernel's buffers hold 16 (token, head) rows
  P.kq_time = n.fold_kq_time; P.ut_time = n.fold_ut_time; P.c_time = n.fold_c_time;
  P.kq_obs = n.fold_kq_obs; P.ut_obs = n.fold_ut_obs; P.c_obs = n.fold_c_obs;
  P.status = c->status;
  P.async_bcast = c->async_bcast ? 1 : 0;
  P.S = c->S;
  P.xt = c->xt; P.xs_b = (long long)(c->cfg.max_K + 1) * c->D;
  P.muhat = c->muhat; P.ms_b = (long long)(c->cfg.max_K > 0 ? c->cfg.max_K : 1) * c->D;
  P.eps = c->eps; P.es_b = P.xs_b;
  P.t = c->t; P.seed = c->seed; P.B = B; P.K = K;
  P.mode = mode; P.C = K + 1;
  P.envp = c->sched_on ? c->envp : nullptr;
  P.item = c->item;
  const bool verify = mode == 1;
  P.resident = (verify ? c->cv_resident : c->dc_resident) ? 1 : 0;
  const int maxc = verify ? c->cv_max_clusters : c->dc_max_clusters, smem = verify ? c->cv_smem : c->dc_smem;
  const int work = verify ? B * (K + 1) : B;
  const int ncl = work < maxc ? work : maxc;
  prof_begin(c, s, verify ? 9 : 7, 0.0);
  if (n.cfg.d == 128) TSDP_LAUNCH(c, (drafter_cluster_kernel<128>), ncl * DC_CS, DC_THREADS, smem, s, P);
  else TSDP_LAUNCH(c, (drafter_cluster_kernel<256>), ncl * DC_CS, DC_THREADS, smem, s, P);
  prof_end(c, s);
  c->launches_per_round_tmp++;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

// ------------------------------------------------------------------------------------------ round
// Enqueue one speculative round for B environments with K draft steps.
int enqueue_round(tsdp_ctx* c, int B, int K, cudaStream_t s, bool dbg) {
  const int D = c->D;
  const long long xs_b = (long long)(c->cfg.max_K + 1) * D, ms_b = (long long)(c->cfg.max_K > 0 ? c->cfg.max_K : 1) * D;
  int r;
  const bool cluster_draft = K > 0 && use_cluster_drafter(c, B);
  const bool cluster_verify = use_cluster_verifier(c, B, K);
  const bool frozen_draft = c->net[TSDP_DRAFT].cfg.arch == TSDP_ARCH_FROZEN;
  // Plan of the round: the layer-by-layer forwards then run on the live candidates only.  Not needed when both sides
  // run in the cluster kernels (small batches), which skip finished slots themselves.
  const bool layered_draft = K > 0 && !cluster_draft && (!frozen_draft || !use_cluster_verifier(c, B, 0));
  const bool compact = c->compact && B <= PLAN_MAX_B && (layered_draft || !cluster_verify);
  if (compact) {
    prof_begin(c, s, 4, 0.0);
    TSDP_LAUNCH(c, (round_plan_kernel), 1, PLAN_THREADS, 0, s, c->t, B, K, c->sched, TSDP_MAX_T + 1, c->round_idx,
                c->sched_on ? c->envp : nullptr, c->item, c->cfg.T, c->plan_live_n, c->plan_list, c->plan_slot_start,
                c->plan_order, c->plan_dn, c->stats);
    prof_end(c, s);
    c->launches_per_round_tmp++;
    CU_TRY(c, cudaGetLastError());
    if (c->prof_on) {      // plain launches, no capture: the counts can be read back for the flop accounting
      CU_TRY(c, cudaStreamSynchronize(s));
      CU_TRY(c, cudaMemcpy(&c->prof_plan_live, c->plan_live_n, sizeof(int), cudaMemcpyDeviceToHost));
      CU_TRY(c, cudaMemcpy(c->prof_plan_dn, c->plan_dn, sizeof(int) * (TSDP_MAX_K + 2), cudaMemcpyDeviceToHost));
    }
  }
  const bool counts_known = compact && c->prof_on;
  if (cluster_draft && (r = launch_cluster_forward(c, TSDP_DRAFT, 0, B, K, s))) return r;
  const float* eps_hat = c->eps_d;        // where the draft step finds eps^ of slot b: eps_hat + b * eps_hat_b
  long long eps_hat_b = D;
  if (frozen_draft && K > 0) {
    // frozen target drafts: the base model's output at the current latent serves every draft step of the round
    if (use_cluster_verifier(c, B, 0)) {          // one cluster per slot; eps lands in candidate slot 0 of the eps buffer
      if ((r = launch_cluster_forward(c, TSDP_BASE, 1, B, 0, s))) return r;
      eps_hat = c->eps; eps_hat_b = xs_b;
    } else {
      CandMap c0{c->xt, xs_b, c->eps_d, (long long)D, c->t, 1, 0, c->item, compact ? c->plan_order : nullptr,
                 compact ? c->plan_dn + 1 : nullptr};      // the slots that draft at all
      c->prof_live_count = counts_known ? c->prof_plan_dn[1] : -1;
      r = forward(c, c->net[TSDP_BASE], c0, B, s);
      c->prof_live_count = -1;
      if (r) return r;
    }
  }
  // transformer drafter, layer by layer: its head, the draft step and the next step's embedding are one kernel
  const bool fused_tail = c->net[TSDP_DRAFT].cfg.arch == TSDP_ARCH_XFMR && c->cfg.A <= 32;
  for (int k = 1; k <= K && !cluster_draft; ++k) {
    CandMap cm{c->xt + (long long)(k - 1) * D, xs_b, c->eps_d, (long long)D, c->t, 1, k - 1, c->item,
               compact ? c->plan_order : nullptr, compact ? c->plan_dn + k : nullptr};     // the slots still drafting at step k
    c->prof_gemm_cat = 6;
    c->xf_skip_embed = fused_tail && k > 1;
    c->xf_skip_head = fused_tail;
    c->prof_live_count = counts_known ? c->prof_plan_dn[k] : -1;
    r = frozen_draft ? TSDP_OK : forward(c, c->net[TSDP_DRAFT], cm, B, s);
    c->prof_live_count = -1;
    c->prof_gemm_cat = 0;
    c->xf_skip_embed = c->xf_skip_head = false;
    if (r) return r;
    if (fused_tail) {
      r = c->cfg.precision == 0 ? draft_tail_launch<float>(c, c->net[TSDP_DRAFT], B, k, K, k < K, s, cm.list, cm.n_live)
                                : draft_tail_launch<__nv_bfloat16>(c, c->net[TSDP_DRAFT], B, k, K, k < K, s, cm.list, cm.n_live);
      if (r) return r;
      continue;
    }
    prof_begin(c, s, 4, 0.0);
    TSDP_LAUNCH(c, (draft_step_kernel), B, 128, 0, s, c->S, c->xt, xs_b, c->muhat, ms_b, eps_hat, eps_hat_b, c->t, k, D, c->seed,
                c->sched_on ? c->envp : nullptr, K, c->cfg.T, c->item);
    prof_end(c, s);
    c->launches_per_round_tmp++;
    CU_TRY(c, cudaGetLastError());
  }
  CandMap cv{c->xt, xs_b, c->eps, xs_b, c->t, K + 1, 0, c->item, compact ? c->plan_list : nullptr,
             compact ? c->plan_live_n : nullptr};
  if (cluster_verify) {
    if ((r = launch_cluster_forward(c, TSDP_BASE, 1, B, K, s))) return r;
  } else {
    c->prof_live_count = counts_known ? c->prof_plan_live : -1;
    r = forward(c, c->net[TSDP_BASE], cv, B * (K + 1), s, c->plan_slot_start);
    c->prof_live_count = -1;
    if (r) return r;
  }
  int warps = K < 1 ? 1 : K;
  if (warps < 4) warps = 4;
  if (warps > 16) warps = 16;
  prof_begin(c, s, 8, 0.0);
  TSDP_LAUNCH(c, (accept_kernel), B, warps * 32, 0, s, c->S, c->xt, xs_b, c->muhat, ms_b, c->eps, xs_b, c->t, K, D, c->seed, c->sched,
                                         TSDP_MAX_T + 1, c->round_idx, c->actions, c->n_done, c->stats, c->cfg.draft_nfe,
                                         dbg ? c->dbg_logalpha : nullptr, dbg ? c->dbg_jstar : nullptr,
                                         c->sched_on ? c->envp : nullptr, c->item, c->queue_head, c->n_items, c->item_counts);
  prof_end(c, s);
  TSDP_LAUNCH(c, (round_end_kernel), 1, 1, 0, s, c->round_idx, c->n_done, c->host_done);
  c->launches_per_round_tmp += 2;
  CU_TRY(c, cudaGetLastError());
  return TSDP_OK;
}

int run_round(tsdp_ctx* c, int B, int K, cudaStream_t s) {
  c->cand_static += (uint64_t)B * (K + 1);
  if (!c->cfg.use_graph || c->prof_on) {
    c->launches_per_round_tmp = 0;
    int r = enqueue_round(c, B, K, s, false);
    c->launches += c->launches_per_round_tmp;
    return r;
  }
  auto key = std::make_tuple(B, K);
  auto it = c->graphs.find(key);
  if (it == c->graphs.end()) {
    // tensor maps must exist before capture; a dry enqueue outside capture would run the round, so
    // instead capture directly: map creation is host-only work and is legal during capture.
    cudaGraph_t graph = nullptr;
    CU_TRY(c, cudaStreamBeginCapture(c->cap_stream, cudaStreamCaptureModeThreadLocal));
    c->launches_per_round_tmp = 0;
    int r = enqueue_round(c, B, K, c->cap_stream, false);
    cudaError_t e = cudaStreamEndCapture(c->cap_stream, &graph);
    if (r != TSDP_OK) { if (graph) cudaGraphDestroy(graph); return r; }
    CU_TRY(c, e);
    cudaGraphExec_t exec = nullptr;
    CU_TRY(c, cudaGraphInstantiate(&exec, graph, 0));
    cudaGraphDestroy(graph);
    it = c->graphs.emplace(key, tsdp_ctx::GraphRec{exec, c->launches_per_round_tmp}).first;
  }
  CU_TRY(c, cudaGraphLaunch(it->second.exec, s));
  c->launches += it->second.launches;
  return TSDP_OK;
}

int check_status(tsdp_ctx* c) {
  int st = 0;
  CU_TRY(c, cudaMemcpy(&st, c->status, sizeof(int), cudaMemcpyDeviceToHost));
  if (st != 0) {
    cudaMemset(c->status, 0, sizeof(int));
    return st;
  }
  return TSDP_OK;
}

void fill_round_params(RoundParams* rp, int K, const tsdp_accept_t& a) {
  rp->K = K;
  rp->mode = a.mode;
  rp->log_lambda = logf(a.lambda > 0.f ? a.lambda : 1e-30f);
  rp->sigma_scale = a.sigma_scale > 0.f ? a.sigma_scale : 1.0f;
  rp->bonus = a.bonus;
}

bool accept_ok(const tsdp_accept_t* a) {
  return a && (a->mode == 0 || a->mode == 1) && a->sigma_scale > 0.f && (a->mode == 0 || (a->lambda > 0.f && a->lambda <= 1.f));
}

// Upload the per-round parameter table: entry r for round r, the last entry repeating.
int upload_schedule(tsdp_ctx* c, int K, const tsdp_accept_t& acc, cudaStream_t s, bool ignore_user_schedule) {
  const int n = ignore_user_schedule ? 0 : (int)c->sched_K.size();
  for (int r = 0; r <= TSDP_MAX_T; ++r) {
    if (n > 0) {
      const int i = r < n ? r : n - 1;
      fill_round_params(&c->sched_host[r], c->sched_K[i], c->sched_acc[i]);
    } else {
      fill_round_params(&c->sched_host[r], K, acc);
    }
  }
  CU_TRY(c, cudaMemcpyAsync(c->sched, c->sched_host, sizeof(RoundParams) * (TSDP_MAX_T + 1), cudaMemcpyHostToDevice, s));
  return TSDP_OK;
}

}  // namespace

// ================================================================================================ C ABI
extern "C" {

const char* tsdp_strerror(int st) {
  switch (st) {
    case TSDP_OK: return "ok";
    case TSDP_ERR_ARG: return "bad argument";
    case TSDP_ERR_STATE: return "weights not loaded";
    case TSDP_ERR_WEIGHTS: return "weight blob does not match the configured architecture";
    case TSDP_ERR_CUDA: return "CUDA call failed";
    case TSDP_ERR_TIMEOUT: return "a bounded wait inside a kernel expired";
    case TSDP_ERR_NAN: return "non-finite value in weights";
    case TSDP_ERR_UNSUPPORTED: return "architecture not built";
    case TSDP_ERR_TOO_LARGE: return "size exceeds the capacity of the built-in scratch array";
    case TSDP_ERR_OVERRUN: return "a kernel wrote past the end of a device buffer";
  }
  return "unknown status";
}

const char* tsdp_last_error(const tsdp_ctx* ctx) { return ctx ? ctx->last_error.c_str() : ""; }

size_t tsdp_weights_count(const tsdp_config_t* cfg, int which) {
  if (cfg && which == TSDP_SCHED) return sched_weights_count(*cfg);
  if (!cfg || (which != TSDP_BASE && which != TSDP_DRAFT)) return 0;
  const tsdp_net_t& n = which == TSDP_BASE ? cfg->base : cfg->draft;
  if (!net_cfg_ok(*cfg, n)) return 0;
  return weights_count(*cfg, n);
}

int tsdp_init(const tsdp_config_t* cfg, tsdp_ctx** out) {
  if (!cfg || !out) return TSDP_ERR_ARG;
  if (cfg->H < 1 || cfg->A < 1 || cfg->T < 1 || cfg->T > TSDP_MAX_T || cfg->max_B < 1 || cfg->max_K < 0 ||
      cfg->max_K > TSDP_MAX_K || cfg->obs_tokens < 0 || cfg->obs_dim < 0 || !(cfg->beta0 > 0.f) || !(cfg->beta1 < 1.f) ||
      (cfg->precision != 0 && cfg->precision != 1) || cfg->drafter < 0 || cfg->drafter > 2 || cfg->verifier < 0 ||
      cfg->verifier > 2)
    return TSDP_ERR_ARG;
  for (const tsdp_net_t* n : {&cfg->base, &cfg->draft}) {
    if (n->arch < TSDP_ARCH_GAUSS || n->arch > TSDP_ARCH_FROZEN) return TSDP_ERR_UNSUPPORTED;
    if (!net_cfg_ok(*cfg, *n)) return TSDP_ERR_ARG;
  }
  tsdp_ctx* c = new tsdp_ctx();
  c->cfg = *cfg;
  c->D = cfg->H * cfg->A;
  c->pdl = getenv("TSDP_NO_PDL") == nullptr;
  c->async_bcast = getenv("TSDP_NO_ASYNC_BCAST") == nullptr;
  c->compact = getenv("TSDP_NO_COMPACT") == nullptr;
  c->no_ksplit = getenv("TSDP_NO_KSPLIT") != nullptr;
  c->tc_attn = getenv("TSDP_NO_TC_ATTN") != nullptr ? 0 : (getenv("TSDP_TC_ATTN") != nullptr ? atoi(getenv("TSDP_TC_ATTN")) : 1);
  if (const char* fb = getenv("TSDP_GEMM_BN")) {      // tuning aid: one tile width for every GEMM it divides
    const int v = atoi(fb);
    if (v == 32 || v == 64 || v == 128 || v == 256) c->force_bn = v;
  }
  auto fail = [&](int st) { tsdp_destroy(c); return st; };
#define INIT_TRY(expr)                                                                    \
  do {                                                                                    \
    cudaError_t e__ = (expr);                                                             \
    if (e__ != cudaSuccess) { fprintf(stderr, "tsdp_init: %s: %s\n", #expr, cudaGetErrorString(e__)); return fail(TSDP_ERR_CUDA); } \
  } while (0)
  INIT_TRY(cudaSetDevice(cfg->device));
  cudaDeviceProp prop;
  INIT_TRY(cudaGetDeviceProperties(&prop, cfg->device));
  c->num_sms = prop.multiProcessorCount;
  if (cfg->precision == 1 && prop.major != 10) {
    fprintf(stderr, "tsdp_init: precision 1 needs an sm_100a device (found sm_%d%d)\n", prop.major, prop.minor);
    return fail(TSDP_ERR_CUDA);
  }
  if (c->cfg.draft_nfe <= 0.f) {
    const int lb = cfg->base.layers, ld = cfg->draft.layers;
    c->cfg.draft_nfe = (lb > 0 && ld > 0) ? (float)ld / (float)lb : 0.125f;
  }
  // DDPM tables (fp64 on the host, stored fp32)
  const int T = cfg->T;
  std::vector<float> tab(5 * T);
  {
    double abar = 1.0, abar_prev = 1.0;
    for (int t = 0; t < T; ++t) {
      const double beta = T > 1 ? cfg->beta0 + ((double)cfg->beta1 - cfg->beta0) * t / (T - 1) : cfg->beta0;
      const double alpha = 1.0 - beta;
      abar_prev = abar;
      abar *= alpha;
      tab[0 * T + t] = (float)std::sqrt(abar);
      tab[1 * T + t] = (float)std::sqrt(1.0 - abar);
      tab[2 * T + t] = (float)(std::sqrt(abar_prev) * beta / (1.0 - abar));
      tab[3 * T + t] = (float)(std::sqrt(alpha) * (1.0 - abar_prev) / (1.0 - abar));
      tab[4 * T + t] = (float)std::sqrt(beta * (1.0 - abar_prev) / (1.0 - abar));
    }
  }
  float* dtab = nullptr;
  if (dev_alloc(c, c->allocs, &dtab, 5 * T)) return fail(TSDP_ERR_CUDA);
  INIT_TRY(cudaMemcpy(dtab, tab.data(), sizeof(float) * 5 * T, cudaMemcpyHostToDevice));
  c->S = DdpmTables{dtab, dtab + T, dtab + 2 * T, dtab + 3 * T, dtab + 4 * T, T, cfg->clip};

  const size_t B = cfg->max_B, K1 = cfg->max_K + 1, Km = cfg->max_K > 0 ? cfg->max_K : 1, D = c->D;
  int st = 0;
  st |= dev_alloc(c, c->allocs, &c->xt, B * K1 * D);
  st |= dev_alloc(c, c->allocs, &c->muhat, B * Km * D);
  st |= dev_alloc(c, c->allocs, &c->eps, B * K1 * D);
  st |= dev_alloc(c, c->allocs, &c->eps_d, B * D);
  st |= dev_alloc(c, c->allocs, &c->actions, B * D);
  st |= dev_alloc(c, c->allocs, &c->obs, B * (size_t)cfg->obs_tokens * cfg->obs_dim + 1);
  st |= dev_alloc(c, c->allocs, &c->t, B);
  st |= dev_alloc(c, c->allocs, &c->seed, 1);
  st |= dev_alloc(c, c->allocs, &c->round_idx, 1);
  st |= dev_alloc(c, c->allocs, &c->n_done, 1);
  st |= dev_alloc(c, c->allocs, &c->status, 1);
  st |= dev_alloc(c, c->allocs, &c->sched, TSDP_MAX_T + 1);
  st |= dev_alloc(c, c->allocs, &c->stats, 1);
  st |= dev_alloc(c, c->allocs, &c->dbg_logalpha, B * Km);
  st |= dev_alloc(c, c->allocs, &c->dbg_jstar, B);
  st |= dev_alloc(c, c->allocs, &c->item, B);
  st |= dev_alloc(c, c->allocs, &c->queue_head, 1);
  st |= dev_alloc(c, c->allocs, &c->n_items, 1);
  c->items_cap = B;
  st |= dev_alloc(c, c->allocs, &c->envp, B);
  st |= dev_alloc(c, c->allocs, &c->progress, B);
  st |= dev_alloc(c, c->allocs, &c->sched_dbg, B * 8);
  st |= dev_alloc(c, c->allocs, &c->item_counts, (size_t)B * 4);
  st |= dev_alloc(c, c->allocs, &c->reward, B);
  st |= dev_alloc(c, c->allocs, &c->plan_live_n, 1);
  st |= dev_alloc(c, c->allocs, &c->plan_list, B * K1);
  st |= dev_alloc(c, c->allocs, &c->plan_slot_start, B + 1);
  st |= dev_alloc(c, c->allocs, &c->plan_order, B);
  st |= dev_alloc(c, c->allocs, &c->plan_dn, TSDP_MAX_K + 2);
  st |= dev_alloc(c, c->allocs, &c->distill_theta, 2);
  st |= dev_alloc(c, c->allocs, &c->distill_terms, 5 * B);
  st |= dev_alloc(c, c->allocs, &c->distill_res, 8);
  if (st) return fail(TSDP_ERR_CUDA);
  INIT_TRY(cudaHostAlloc(reinterpret_cast<void**>(&c->host_done), sizeof(int), cudaHostAllocMapped));
  *c->host_done = 0;
  INIT_TRY(cudaHostAlloc(reinterpret_cast<void**>(&c->sched_host), sizeof(RoundParams) * (TSDP_MAX_T + 1), cudaHostAllocDefault));
  INIT_TRY(cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking));
  INIT_TRY(cudaStreamCreateWithFlags(&c->side_stream, cudaStreamNonBlocking));
  INIT_TRY(cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming));
  INIT_TRY(cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming));
  INIT_TRY(cudaStreamCreateWithFlags(&c->aux_stream, cudaStreamNonBlocking));
  INIT_TRY(cudaEventCreateWithFlags(&c->ev_aux_fork, cudaEventDisableTiming));
  INIT_TRY(cudaEventCreateWithFlags(&c->ev_aux_join, cudaEventDisableTiming));
  c->aux_on = getenv("TSDP_NO_AUX_STREAM") == nullptr;
  INIT_TRY(cudaEventCreate(&c->ev_chunk0));
  INIT_TRY(cudaEventCreate(&c->ev_chunk1));
  c->lat_ring.assign(TSDP_LATENCY_RING, 0.f);

  // transformer workspaces, sized for the larger of (base over all candidates, drafter over B)
  size_t rows_d = 0, rows_4d = 0, mem_rows_d = 0;
  const int esz = cfg->precision == 0 ? 4 : 2;
  for (int w = 0; w < 2; ++w) {
    const tsdp_net_t& n = w == TSDP_BASE ? cfg->base : cfg->draft;
    if (n.arch != TSDP_ARCH_XFMR && n.arch != TSDP_ARCH_DIT) continue;
    const size_t M = (w == TSDP_BASE ? B * K1 : B) * cfg->H;
    rows_d = std::max(rows_d, M * n.d);
    rows_4d = std::max(rows_4d, M * 4 * n.d);
    mem_rows_d = std::max(mem_rows_d, std::max((size_t)T, B * cfg->obs_tokens) * n.d);
  }
  if (rows_d) {
    st |= dev_alloc(c, c->allocs, &c->h, rows_d);
    st |= alloc_bytes(c, c->allocs, &c->a, rows_d * esz);
    st |= alloc_bytes(c, c->allocs, &c->qkv, rows_d * 3 * esz);
    st |= alloc_bytes(c, c->allocs, &c->q2, rows_d * esz);
    st |= alloc_bytes(c, c->allocs, &c->f, rows_4d * esz);
    st |= alloc_bytes(c, c->allocs, &c->memtok, mem_rows_d * esz);
    if (st) return fail(TSDP_ERR_CUDA);
  }
  if (cfg->precision == 1) {
    cudaDriverEntryPointQueryResult q;
    void* fn = nullptr;
    INIT_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
    if (!fn || q != cudaDriverEntryPointSuccess) { fprintf(stderr, "tsdp_init: cuTensorMapEncodeTiled unavailable\n"); return fail(TSDP_ERR_CUDA); }
    c->encode = reinterpret_cast<EncodeTiledFn>(fn);
    INIT_TRY(set_smem_attr_all<256>());
    INIT_TRY(set_smem_attr_all<128>());
    INIT_TRY(set_smem_attr_all<64>());
    INIT_TRY(set_smem_attr_all<32>());
    INIT_TRY(cudaFuncSetAttribute(gemm_tcgen05_kernel<GEMM_ATTN_BN, EPI_ATTN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  gemm_smem_bytes(GEMM_ATTN_BN)));
    if (const char* pm = getenv("TSDP_GEMM_PAIR")) c->pair_mode = atoi(pm);
    if (c->pair_mode != 0) {      // CTA-pair kernels: shared-memory opt-in and how many clusters of 2 the device holds at once
      const void* fns[6] = {(const void*)gemm_tcgen05_kernel<256, EPI_STORE, 2>, (const void*)gemm_tcgen05_kernel<256, EPI_GELU, 2>,
                            (const void*)gemm_tcgen05_kernel<256, EPI_RESID, 2>, (const void*)gemm_tcgen05_kernel<256, EPI_GATE, 2>,
                            (const void*)gemm_tcgen05_kernel<256, EPI_F32, 2>, (const void*)gemm_tcgen05_kernel<GEMM_ATTN_BN, EPI_ATTN, 2>};
      for (int i = 0; i < 6; ++i) {
        const int smem = i < 5 ? gemm_smem_bytes_cg(256, 2) : gemm_smem_bytes_cg(GEMM_ATTN_BN, 2);
        INIT_TRY(cudaFuncSetAttribute(fns[i], cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        if (i != 0 && i != 5) continue;
        cudaLaunchConfig_t lc{};
        lc.gridDim = dim3(2 * c->num_sms); lc.blockDim = dim3(GEMM_THREADS); lc.dynamicSmemBytes = (size_t)smem;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        lc.attrs = at; lc.numAttrs = 1;
        int ncl = 0;
        if (cudaOccupancyMaxActiveClusters(&ncl, fns[i], &lc) != cudaSuccess) { cudaGetLastError(); ncl = 0; }
        if (i == 0) c->pair_clusters = ncl; else c->pair_clusters_attn = ncl;
      }
      if (getenv("TSDP_VERBOSE"))
        fprintf(stderr, "tsdp_init: CTA-pair GEMM mode %d, %d / %d co-resident clusters of 2\n", c->pair_mode, c->pair_clusters,
                c->pair_clusters_attn);
    }
  }
  for (int which = 0; which < 2; ++which) {
    const tsdp_net_t& nn = which == TSDP_BASE ? cfg->base : cfg->draft;
    int smem = 0; bool res = false;
    if (!cluster_drafter_fits(*cfg, nn, &smem, &res)) continue;
    const void* fn = nn.d == 128 ? (const void*)drafter_cluster_kernel<128> : (const void*)drafter_cluster_kernel<256>;
    int cur_attr = 0;   // both nets may use the same instantiation: keep the larger request
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, fn) == cudaSuccess) cur_attr = fa.maxDynamicSharedSizeBytes;
    if (smem > cur_attr) INIT_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(DC_CS * 64); lc.blockDim = dim3(DC_THREADS); lc.dynamicSmemBytes = (size_t)smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = DC_CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    lc.attrs = at; lc.numAttrs = 1;
    int ncl = 0;
    if (cudaOccupancyMaxActiveClusters(&ncl, fn, &lc) != cudaSuccess || ncl < 1) { cudaGetLastError(); ncl = 0; }
    if (which == TSDP_DRAFT) { c->dc_smem = smem; c->dc_resident = res; c->dc_max_clusters = ncl; c->dc_ok = ncl >= 1; }
    else { c->cv_smem = smem; c->cv_resident = res; c->cv_max_clusters = ncl; c->cv_ok = ncl >= 1; }
  }
  if (cfg->verifier == 2 && !c->cv_ok) {
    fprintf(stderr, "tsdp_init: the cluster verification kernel does not fit this configuration\n");
    return fail(TSDP_ERR_UNSUPPORTED);
  }
  if (cfg->drafter == 2 && !c->dc_ok) {
    fprintf(stderr, "tsdp_init: the persistent cluster drafter does not fit this configuration\n");
    return fail(TSDP_ERR_UNSUPPORTED);
  }
  INIT_TRY(cudaFuncSetAttribute(cross_attn_ctx_mma_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, cx_smem_bytes<32>(256)));
  INIT_TRY(cudaFuncSetAttribute(cross_attn_ctx_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, cx_smem_bytes<64>(256)));
  INIT_TRY(cudaFuncSetAttribute(cross_attn_ctx_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, cx_smem_bytes<128>(256)));
  INIT_TRY(cudaFuncSetAttribute(cross_attn_ctx_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, CXT_SMEM_BYTES));
  INIT_TRY(cudaFuncSetAttribute(xfold_build_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
  INIT_TRY(cudaFuncSetAttribute(xattn_fold_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)xf_smem_bytes(128, XF_MAXN)));
  INIT_TRY(cudaFuncSetAttribute(xattn_fold_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)xf_smem_bytes(256, XF_MAXN)));
  INIT_TRY(cudaFuncSetAttribute(xattn_fold_kernel<512>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)xf_smem_bytes(512, XF_MAXN)));
  INIT_TRY(cudaFuncSetAttribute(self_attn_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
  INIT_TRY(cudaFuncSetAttribute(self_attn_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
  c->net[TSDP_BASE].cfg = cfg->base;
  c->net[TSDP_DRAFT].cfg = cfg->draft;
  if (cfg->draft.arch == TSDP_ARCH_FROZEN) {      // nothing to load; its drafts cost a base forward per round, not drafter calls
    c->net[TSDP_DRAFT].loaded = true;
    c->cfg.draft_nfe = 0.f;
  }
  for (int w = 0; w < 2; ++w) {      // conv-UNet activations: one zero-padded tensor per named stage
    Net& n = c->net[w];
    if (n.cfg.arch != TSDP_ARCH_UNET) continue;
    const size_t nc = (w == TSDP_BASE ? B * K1 : B), ch = n.cfg.d, LV = n.cfg.layers, last = LV - 1;
    auto pad = [&](void** p, size_t lv, size_t C) { return alloc_bytes(c, c->allocs, p, nc * ((cfg->H >> lv) + 4) * C * esz); };
    int e = 0;
    e |= pad(&n.uw.X0, 0, ch); e |= pad(&n.uw.HB, 0, ch);
    e |= pad(&n.uw.E, last, ch << last); e |= pad(&n.uw.M1, last, ch << last); e |= pad(&n.uw.M2, last, ch << last);
    for (size_t lv = 0; lv < LV; ++lv) {
      e |= pad(&n.uw.TMP[lv], lv, ch << lv); e |= pad(&n.uw.D[lv], lv, ch << lv);
      if (lv < last) {
        e |= pad(&n.uw.CAT[lv], lv, (ch << (lv + 1)) + (ch << lv)); e |= pad(&n.uw.P[lv], lv + 1, ch << lv);
        e |= pad(&n.uw.U1[lv], lv, ch << lv); e |= pad(&n.uw.U2[lv], lv, ch << lv);
      }
    }
    n.uw.Y_cap = 4 * nc * (cfg->H + 4) * (ch << last);      // room for the partial sums of a split reduction (conv_ksplit)
    e |= dev_alloc(c, c->allocs, &n.uw.Y, n.uw.Y_cap);
    e |= dev_alloc(c, c->allocs, &n.uw.R, nc * (cfg->H + 4) * (ch << last));
    if (e) return fail(TSDP_ERR_CUDA);
  }
  INIT_TRY(cudaDeviceSynchronize());
#undef INIT_TRY
  *out = c;
  return TSDP_OK;
}

void tsdp_destroy(tsdp_ctx* c) {
  if (!c) return;
  cudaSetDevice(c->cfg.device);
  cudaDeviceSynchronize();
  for (auto& g : c->graphs) cudaGraphExecDestroy(g.second.exec);
  for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
  dev_free_pool(c, c->allocs);
  for (int w = 0; w < 2; ++w) dev_free_pool(c, c->net[w].allocs);
  if (c->host_done) cudaFreeHost(c->host_done);
  if (c->sched_host) cudaFreeHost(c->sched_host);
  if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
  if (c->side_stream) cudaStreamDestroy(c->side_stream);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_join) cudaEventDestroy(c->ev_join);
  if (c->ev_aux_fork) cudaEventDestroy(c->ev_aux_fork);
  if (c->ev_aux_join) cudaEventDestroy(c->ev_aux_join);
  if (c->aux_stream) cudaStreamDestroy(c->aux_stream);
  if (c->ev_chunk0) cudaEventDestroy(c->ev_chunk0);
  if (c->ev_chunk1) cudaEventDestroy(c->ev_chunk1);
  dev_free_pool(c, c->sched_allocs);
  delete c;
}

static int load_sched_weights(tsdp_ctx* c, const float* blob, size_t n) {
  if (n != sched_weights_count(c->cfg)) return TSDP_ERR_WEIGHTS;
  for (size_t i = 0; i < n; ++i)
    if (!std::isfinite(blob[i])) return TSDP_ERR_NAN;
  CU_TRY(c, cudaDeviceSynchronize());
  dev_free_pool(c, c->sched_allocs);
  c->sched_loaded = false;
  float* d = nullptr;
  if (dev_alloc(c, c->sched_allocs, &d, n)) return TSDP_ERR_CUDA;
  CU_TRY(c, cudaMemcpy(d, blob, n * sizeof(float), cudaMemcpyHostToDevice));
  const size_t obs_len = (size_t)c->cfg.obs_tokens * c->cfg.obs_dim, D = c->D;
  SchedWeights& w = c->sched_w;
  w.W_o = d; d += obs_len * SCHED_HID; w.b_o = d; d += SCHED_HID;
  w.W_a = d; d += D * SCHED_HID; w.b_a = d; d += SCHED_HID;
  w.W_p = d; d += SCHED_PROG; w.b_p = d; d += SCHED_PROG;
  w.W_1 = d; d += (size_t)SCHED_CAT * SCHED_HID; w.b_1 = d; d += SCHED_HID;
  w.W_2 = d; d += (size_t)SCHED_HID * SCHED_OUT; w.b_2 = d;
  c->sched_loaded = true;
  return TSDP_OK;
}

int tsdp_load_weights(tsdp_ctx* c, int which, const float* blob, size_t n) {
  if (c && blob && which == TSDP_SCHED) {
    CU_TRY(c, cudaSetDevice(c->cfg.device));
    return load_sched_weights(c, blob, n);
  }
  if (!c || !blob || (which != TSDP_BASE && which != TSDP_DRAFT)) return TSDP_ERR_ARG;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  Net& net = c->net[which];
  const tsdp_config_t& cfg = c->cfg;
  if (net.cfg.arch == TSDP_ARCH_FROZEN) return TSDP_ERR_ARG;      // frozen target drafts have no weights
  if (n != weights_count(cfg, net.cfg)) return TSDP_ERR_WEIGHTS;
  for (size_t i = 0; i < n; ++i)
    if (!std::isfinite(blob[i])) return TSDP_ERR_NAN;
  CU_TRY(c, cudaDeviceSynchronize());
  dev_free_pool(c, net.allocs);
  net.L.clear();
  net.loaded = false;
  // graphs captured with the old pointers are stale
  for (auto& g : c->graphs) cudaGraphExecDestroy(g.second.exec);
  c->graphs.clear();
  c->maps.clear();

  const float* cur = blob;
  const int D = c->D, T = cfg.T;
  auto up_f32 = [&](float** dst, size_t cnt) -> int {
    if (dev_alloc(c, net.allocs, dst, cnt)) return TSDP_ERR_CUDA;
    CU_TRY(c, cudaMemcpy(*dst, cur, cnt * sizeof(float), cudaMemcpyHostToDevice));
    cur += cnt;
    return TSDP_OK;
  };
  // W [in, out] in the blob -> [out, in] on the device, in the GEMM operand type
  auto up_wT = [&](void** dst, const float* src, size_t in, size_t outn) -> int {
    if (cfg.precision == 0) {
      std::vector<float> tmp(in * outn);
      for (size_t i = 0; i < in; ++i)
        for (size_t o = 0; o < outn; ++o) tmp[o * in + i] = src[i * outn + o];
      float* p;
      if (dev_alloc(c, net.allocs, &p, in * outn)) return TSDP_ERR_CUDA;
      CU_TRY(c, cudaMemcpy(p, tmp.data(), tmp.size() * sizeof(float), cudaMemcpyHostToDevice));
      *dst = p;
    } else {
      std::vector<__nv_bfloat16> tmp(in * outn);
      for (size_t i = 0; i < in; ++i)
        for (size_t o = 0; o < outn; ++o) tmp[o * in + i] = __float2bfloat16_rn(src[i * outn + o]);
      __nv_bfloat16* p;
      if (dev_alloc(c, net.allocs, &p, in * outn)) return TSDP_ERR_CUDA;
      CU_TRY(c, cudaMemcpy(p, tmp.data(), tmp.size() * sizeof(__nv_bfloat16), cudaMemcpyHostToDevice));
      *dst = p;
    }
    return TSDP_OK;
  };
  auto sinus_table = [&](int dim, float** dst) -> int {
    std::vector<float> tb((size_t)T * dim);
    const int half = dim / 2;
    for (int t = 0; t < T; ++t)
      for (int i = 0; i < half; ++i) {
        const double fr = std::pow(10000.0, -(double)i / half);
        tb[(size_t)t * dim + i] = (float)std::sin(t * fr);
        tb[(size_t)t * dim + half + i] = (float)std::cos(t * fr);
      }
    if (dev_alloc(c, net.allocs, dst, tb.size())) return TSDP_ERR_CUDA;
    CU_TRY(c, cudaMemcpy(*dst, tb.data(), tb.size() * sizeof(float), cudaMemcpyHostToDevice));
    return TSDP_OK;
  };
  int r;
  if (net.cfg.arch == TSDP_ARCH_GAUSS) {
    net.m0 = blob[0];
    net.s0 = blob[1];
  } else if (net.cfg.arch == TSDP_ARCH_MLP) {
    MlpWeights& m = net.mlp;
    m = MlpWeights{};
    m.n_lin = net.cfg.layers + 1;
    m.temb = net.cfg.temb;
    m.dims[0] = D + net.cfg.temb + cfg.obs_tokens * cfg.obs_dim;
    for (int l = 1; l <= net.cfg.layers; ++l) m.dims[l] = net.cfg.d;
    m.dims[m.n_lin] = D;
    for (int l = 0; l < m.n_lin; ++l) {
      float *W, *b;
      if ((r = up_f32(&W, (size_t)m.dims[l] * m.dims[l + 1]))) return r;
      if ((r = up_f32(&b, m.dims[l + 1]))) return r;
      m.W[l] = W; m.b[l] = b;
    }
    float* tt;
    if ((r = sinus_table(net.cfg.temb, &tt))) return r;
    m.temb_table = tt;
  } else if (net.cfg.arch == TSDP_ARCH_UNET) {
    const size_t ch = net.cfg.d, A = cfg.A, dt = net.cfg.temb, dobs = (size_t)cfg.obs_tokens * cfg.obs_dim, dc = dt + dobs;
    if ((r = up_f32(&net.W_in, A * ch))) return r;
    if ((r = up_f32(&net.b_in, ch))) return r;
    const float *Wt1 = cur, *bt1 = Wt1 + dt * 4 * dt, *Wt2 = bt1 + 4 * dt, *bt2 = Wt2 + 4 * dt * dt;
    cur = bt2 + dt;
    const auto chans = unet_channels((int)ch, net.cfg.layers);
    size_t F = 0;
    for (auto& cc : chans) F += 2 * (size_t)cc.second;
    net.F = (int)F;
    std::vector<float> wfT_time(F * dt), wfT_obs(F * (dobs ? dobs : 1)), bf_all(F);
    net.ub.clear();
    size_t foff = 0;
    for (auto& cc : chans) {
      Net::UBlock b{};
      const size_t ci = cc.first, co = cc.second;
      b.cin = (int)ci; b.cout = (int)co; b.foff = (int)foff;
      if ((r = up_wT(&b.W1, cur, 5 * ci, co))) return r;
      cur += 5 * ci * co;
      if ((r = up_f32(&b.b1, co))) return r;
      if ((r = up_f32(&b.g1, co))) return r;
      if ((r = up_f32(&b.be1, co))) return r;
      for (size_t i = 0; i < dc; ++i)                       // Wf [dc, 2co] -> rows foff.. of the [F, dt] and [F, dobs] tables
        for (size_t o = 0; o < 2 * co; ++o) {
          const float v = cur[i * 2 * co + o];
          if (i < dt) wfT_time[(foff + o) * dt + i] = v; else wfT_obs[(foff + o) * dobs + (i - dt)] = v;
        }
      cur += dc * 2 * co;
      for (size_t o = 0; o < 2 * co; ++o) bf_all[foff + o] = cur[o];
      cur += 2 * co;
      if ((r = up_wT(&b.W2, cur, 5 * co, co))) return r;
      cur += 5 * co * co;
      if ((r = up_f32(&b.b2, co))) return r;
      if ((r = up_f32(&b.g2, co))) return r;
      if ((r = up_f32(&b.be2, co))) return r;
      if (ci != co) {
        if ((r = up_wT(&b.Wr, cur, ci, co))) return r;
        cur += ci * co;
        if ((r = up_f32(&b.br, co))) return r;
      }
      foff += 2 * co;
      net.ub.push_back(b);
    }
    if ((r = up_wT(&net.Wh, cur, 5 * ch, ch))) return r;
    cur += 5 * ch * ch;
    if ((r = up_f32(&net.bh, ch))) return r;
    if ((r = up_f32(&net.gh, ch))) return r;
    if ((r = up_f32(&net.beh, ch))) return r;
    {   // W_out [ch, A] -> fp32 [A, ch]
      std::vector<float> tmp(A * ch);
      for (size_t i = 0; i < ch; ++i)
        for (size_t a = 0; a < A; ++a) tmp[a * ch + i] = cur[i * A + a];
      cur += ch * A;
      if (dev_alloc(c, net.allocs, &net.W_outT, A * ch)) return TSDP_ERR_CUDA;
      CU_TRY(c, cudaMemcpy(net.W_outT, tmp.data(), tmp.size() * sizeof(float), cudaMemcpyHostToDevice));
    }
    if ((r = up_f32(&net.b_out, A))) return r;
    if (dev_alloc(c, net.allocs, &net.film_time, (size_t)T * F)) return TSDP_ERR_CUDA;
    if (dev_alloc(c, net.allocs, &net.film_obs, c->items_cap * F)) return TSDP_ERR_CUDA;
    if (dev_alloc(c, net.allocs, &net.obs_m, c->items_cap * (dobs ? dobs : 1))) return TSDP_ERR_CUDA;
    if (dev_alloc(c, net.allocs, &net.WfT_obs, F * (dobs ? dobs : 1))) return TSDP_ERR_CUDA;
    CU_TRY(c, cudaMemcpy(net.WfT_obs, wfT_obs.data(), wfT_obs.size() * sizeof(float), cudaMemcpyHostToDevice));
    if ((r = sinus_table((int)dt, &net.temb_table))) return r;
    // time vector for every t, then its FiLM contribution: film_time = Mish(tvec) Wf_time + bf
    std::vector<float> wt1T(4 * dt * dt), wt2T(dt * 4 * dt);
    for (size_t i = 0; i < dt; ++i)
      for (size_t o = 0; o < 4 * dt; ++o) wt1T[o * dt + i] = Wt1[i * 4 * dt + o];
    for (size_t i = 0; i < 4 * dt; ++i)
      for (size_t o = 0; o < dt; ++o) wt2T[o * 4 * dt + i] = Wt2[i * dt + o];
    std::vector<void*> tmp_pool;
    float *d_w1, *d_b1, *d_w2, *d_b2, *d_wf, *d_bf, *d_hid, *d_tv;
    int st = 0;
    st |= dev_alloc(c, tmp_pool, &d_w1, 4 * dt * dt); st |= dev_alloc(c, tmp_pool, &d_b1, 4 * dt);
    st |= dev_alloc(c, tmp_pool, &d_w2, 4 * dt * dt); st |= dev_alloc(c, tmp_pool, &d_b2, dt);
    st |= dev_alloc(c, tmp_pool, &d_wf, F * dt); st |= dev_alloc(c, tmp_pool, &d_bf, F);
    st |= dev_alloc(c, tmp_pool, &d_hid, (size_t)T * 4 * dt); st |= dev_alloc(c, tmp_pool, &d_tv, (size_t)T * dt);
    auto free_tmp = [&]() { dev_free_pool(c, tmp_pool); };
    if (st) { free_tmp(); return TSDP_ERR_CUDA; }
    cudaMemcpy(d_w1, wt1T.data(), wt1T.size() * 4, cudaMemcpyHostToDevice); cudaMemcpy(d_b1, bt1, 4 * dt * 4, cudaMemcpyHostToDevice);
    cudaMemcpy(d_w2, wt2T.data(), wt2T.size() * 4, cudaMemcpyHostToDevice); cudaMemcpy(d_b2, bt2, dt * 4, cudaMemcpyHostToDevice);
    cudaMemcpy(d_wf, wfT_time.data(), wfT_time.size() * 4, cudaMemcpyHostToDevice);
    cudaMemcpy(d_bf, bf_all.data(), F * 4, cudaMemcpyHostToDevice);
    r = gemm_f32(c, net.temb_table, d_w1, d_b1, T, (int)(4 * dt), (int)dt, EPI_MISH, d_hid, 0);
    if (!r) r = gemm_f32(c, d_hid, d_w2, d_b2, T, (int)dt, (int)(4 * dt), EPI_F32, d_tv, 0);
    if (!r) {
      const long long nel = (long long)T * dt;
      mish_kernel<<<(unsigned)((nel + 255) / 256), 256>>>(d_tv, d_tv, nel);
      r = gemm_f32(c, d_tv, d_wf, d_bf, T, (int)F, (int)dt, EPI_F32, net.film_time, 0);
    }
    cudaError_t e = cudaDeviceSynchronize();
    free_tmp();
    if (r) return r;
    CU_TRY(c, e);
  } else if (net.cfg.arch == TSDP_ARCH_DIT) {
    const size_t d = net.cfg.d, A = cfg.A, H = cfg.H, Tc = cfg.obs_tokens, L = net.cfg.layers;
    if ((r = up_f32(&net.W_in, A * d))) return r;
    if ((r = up_f32(&net.b_in, d))) return r;
    if ((r = up_f32(&net.pos, H * d))) return r;
    if ((r = up_f32(&net.W_obs, (size_t)cfg.obs_dim * d))) return r;
    if ((r = up_f32(&net.b_obs, d))) return r;
    if ((r = up_f32(&net.cpos, Tc * d))) return r;
    // time path and modulation layers stay fp32: they only feed tables built below
    const float *Wt1 = cur, *bt1 = cur + d * d, *Wt2 = bt1 + d, *bt2 = Wt2 + d * d;
    cur = bt2 + d;
    const size_t mod_ld = L * 6 * d + 2 * d;
    std::vector<float> wmodT(mod_ld * d), bmod(mod_ld);          // [out = L*6d + 2d, in = d]
    std::vector<float> wkv_all(d * L * 2 * d), bkv_all(L * 2 * d);
    net.L.resize(L);
    for (size_t l = 0; l < L; ++l) {
      XfmrLayer& w = net.L[l];
      for (size_t i = 0; i < d; ++i)
        for (size_t o = 0; o < 6 * d; ++o) wmodT[(l * 6 * d + o) * d + i] = cur[i * 6 * d + o];
      cur += d * 6 * d;
      for (size_t o = 0; o < 6 * d; ++o) bmod[l * 6 * d + o] = cur[o];
      cur += 6 * d;
      if ((r = up_wT(&w.Wqkv, cur, d, 3 * d))) return r;
      cur += d * 3 * d;
      if ((r = up_f32(&w.bqkv, 3 * d))) return r;
      if ((r = up_wT(&w.Wo, cur, d, d))) return r;
      cur += d * d;
      if ((r = up_f32(&w.bo, d))) return r;
      if ((r = up_f32(&w.ln2_g, d))) return r;
      if ((r = up_f32(&w.ln2_b, d))) return r;
      if ((r = up_wT(&w.Wq2, cur, d, d))) return r;
      cur += d * d;
      if ((r = up_f32(&w.bq2, d))) return r;
      for (size_t i = 0; i < d; ++i)
        for (size_t o = 0; o < 2 * d; ++o) wkv_all[i * (L * 2 * d) + l * 2 * d + o] = cur[i * 2 * d + o];
      cur += d * 2 * d;
      for (size_t o = 0; o < 2 * d; ++o) bkv_all[l * 2 * d + o] = cur[o];
      cur += 2 * d;
      if ((r = up_wT(&w.Wo2, cur, d, d))) return r;
      cur += d * d;
      if ((r = up_f32(&w.bo2, d))) return r;
      if ((r = up_wT(&w.W1, cur, d, 4 * d))) return r;
      cur += d * 4 * d;
      if ((r = up_f32(&w.b1, 4 * d))) return r;
      if ((r = up_wT(&w.W2, cur, 4 * d, d))) return r;
      cur += 4 * d * d;
      if ((r = up_f32(&w.b2, d))) return r;
    }
    for (size_t i = 0; i < d; ++i)
      for (size_t o = 0; o < 2 * d; ++o) wmodT[(L * 6 * d + o) * d + i] = cur[i * 2 * d + o];
    cur += d * 2 * d;
    for (size_t o = 0; o < 2 * d; ++o) bmod[L * 6 * d + o] = cur[o];
    cur += 2 * d;
    {   // W_out [d, A] -> fp32 [A, d]
      std::vector<float> tmp(A * d);
      for (size_t i = 0; i < d; ++i)
        for (size_t a = 0; a < A; ++a) tmp[a * d + i] = cur[i * A + a];
      cur += d * A;
      if (dev_alloc(c, net.allocs, &net.W_outT, A * d)) return TSDP_ERR_CUDA;
      CU_TRY(c, cudaMemcpy(net.W_outT, tmp.data(), tmp.size() * sizeof(float), cudaMemcpyHostToDevice));
    }
    if ((r = up_f32(&net.b_out, A))) return r;
    if ((r = up_wT(&net.Wkv_all, wkv_all.data(), d, L * 2 * d))) return r;
    if (dev_alloc(c, net.allocs, &net.bkv_all, L * 2 * d)) return TSDP_ERR_CUDA;
    CU_TRY(c, cudaMemcpy(net.bkv_all, bkv_all.data(), bkv_all.size() * sizeof(float), cudaMemcpyHostToDevice));
    if (dev_alloc(c, net.allocs, &net.kv_obs, c->items_cap * Tc * L * 2 * d)) return TSDP_ERR_CUDA;
    if ((r = sinus_table((int)d, &net.temb_table))) return r;
    // Tables of the timestep path, for every t: c = W_t2^T SiLU(W_t1^T sin(t) + b_t1) + b_t2, then every block's
    // (shift, scale, gate) vectors and the final layer's = SiLU(c) W_mod + b_mod.
    if (dev_alloc(c, net.allocs, &net.mod, (size_t)T * mod_ld)) return TSDP_ERR_CUDA;
    net.mod_ld = (int)mod_ld;
    std::vector<float> wt1T(d * d), wt2T(d * d);
    for (size_t i = 0; i < d; ++i)
      for (size_t o = 0; o < d; ++o) { wt1T[o * d + i] = Wt1[i * d + o]; wt2T[o * d + i] = Wt2[i * d + o]; }
    std::vector<void*> tmp_pool;
    float *d_w1, *d_b1, *d_w2, *d_b2, *d_wm, *d_bm, *d_hid, *d_c;
    int st = 0;
    st |= dev_alloc(c, tmp_pool, &d_w1, d * d); st |= dev_alloc(c, tmp_pool, &d_b1, d);
    st |= dev_alloc(c, tmp_pool, &d_w2, d * d); st |= dev_alloc(c, tmp_pool, &d_b2, d);
    st |= dev_alloc(c, tmp_pool, &d_wm, mod_ld * d); st |= dev_alloc(c, tmp_pool, &d_bm, mod_ld);
    st |= dev_alloc(c, tmp_pool, &d_hid, (size_t)T * d); st |= dev_alloc(c, tmp_pool, &d_c, (size_t)T * d);
    auto free_tmp = [&]() { dev_free_pool(c, tmp_pool); };
    if (st) { free_tmp(); return TSDP_ERR_CUDA; }
    cudaMemcpy(d_w1, wt1T.data(), d * d * 4, cudaMemcpyHostToDevice); cudaMemcpy(d_b1, bt1, d * 4, cudaMemcpyHostToDevice);
    cudaMemcpy(d_w2, wt2T.data(), d * d * 4, cudaMemcpyHostToDevice); cudaMemcpy(d_b2, bt2, d * 4, cudaMemcpyHostToDevice);
    cudaMemcpy(d_wm, wmodT.data(), mod_ld * d * 4, cudaMemcpyHostToDevice);
    cudaMemcpy(d_bm, bmod.data(), mod_ld * 4, cudaMemcpyHostToDevice);
    r = gemm_f32(c, net.temb_table, d_w1, d_b1, T, (int)d, (int)d, EPI_SILU, d_hid, 0);
    if (!r) r = gemm_f32(c, d_hid, d_w2, d_b2, T, (int)d, (int)d, EPI_F32, d_c, 0);
    if (!r) {
      const long long nel = (long long)T * d;
      silu_inplace_kernel<<<(unsigned)((nel + 255) / 256), 256>>>(d_c, nel);
      r = gemm_f32(c, d_c, d_wm, d_bm, T, (int)mod_ld, (int)d, EPI_F32, net.mod, 0);
    }
    cudaError_t e = cudaDeviceSynchronize();
    free_tmp();
    if (r) return r;
    CU_TRY(c, e);
  } else {
    const size_t d = net.cfg.d, A = cfg.A, H = cfg.H, To = cfg.obs_tokens, L = net.cfg.layers;
    if ((r = up_f32(&net.W_in, A * d))) return r;
    if ((r = up_f32(&net.b_in, d))) return r;
    if ((r = up_f32(&net.pos, H * d))) return r;
    if ((r = up_f32(&net.W_obs, (size_t)cfg.obs_dim * d))) return r;
    if ((r = up_f32(&net.b_obs, d))) return r;
    if ((r = up_f32(&net.cpos, (1 + To) * d))) return r;
    std::vector<float> wkv_all(d * L * 2 * d), bkv_all(L * 2 * d);   // [in = d, out = L*2d]
    net.L.resize(L);
    for (size_t l = 0; l < L; ++l) {
      XfmrLayer& w = net.L[l];
      if ((r = up_f32(&w.ln1_g, d))) return r;
      if ((r = up_f32(&w.ln1_b, d))) return r;
      if ((r = up_wT(&w.Wqkv, cur, d, 3 * d))) return r;
      if (fused_attn_ok(cfg, net.cfg)) {      // the same matrix and bias, output features head-major
        std::vector<float> wp(d * 3 * d), bp(3 * d);
        const float* bsrc = cur + d * 3 * d;
        for (size_t o = 0; o < 3 * d; ++o) {
          const size_t which = o / d, hd = (o % d) / 64, cc = o % 64, on = hd * 192 + which * 64 + cc;
          for (size_t i = 0; i < d; ++i) wp[i * 3 * d + on] = cur[i * 3 * d + o];
          bp[on] = bsrc[o];
        }
        if ((r = up_wT(&w.Wqkv_hm, wp.data(), d, 3 * d))) return r;
        if (dev_alloc(c, net.allocs, &w.bqkv_hm, 3 * d)) return TSDP_ERR_CUDA;
        CU_TRY(c, cudaMemcpy(w.bqkv_hm, bp.data(), 3 * d * sizeof(float), cudaMemcpyHostToDevice));
      }
      cur += d * 3 * d;
      if ((r = up_f32(&w.bqkv, 3 * d))) return r;
      if ((r = up_wT(&w.Wo, cur, d, d))) return r;
      cur += d * d;
      if ((r = up_f32(&w.bo, d))) return r;
      if ((r = up_f32(&w.ln2_g, d))) return r;
      if ((r = up_f32(&w.ln2_b, d))) return r;
      if ((r = up_wT(&w.Wq2, cur, d, d))) return r;
      cur += d * d;
      if ((r = up_f32(&w.bq2, d))) return r;
      for (size_t i = 0; i < d; ++i)
        for (size_t o = 0; o < 2 * d; ++o) wkv_all[i * (L * 2 * d) + l * 2 * d + o] = cur[i * 2 * d + o];
      cur += d * 2 * d;
      for (size_t o = 0; o < 2 * d; ++o) bkv_all[l * 2 * d + o] = cur[o];
      cur += 2 * d;
      if ((r = up_wT(&w.Wo2, cur, d, d))) return r;
      cur += d * d;
      if ((r = up_f32(&w.bo2, d))) return r;
      if ((r = up_f32(&w.ln3_g, d))) return r;
      if ((r = up_f32(&w.ln3_b, d))) return r;
      if ((r = up_wT(&w.W1, cur, d, 4 * d))) return r;
      cur += d * 4 * d;
      if ((r = up_f32(&w.b1, 4 * d))) return r;
      if ((r = up_wT(&w.W2, cur, 4 * d, d))) return r;
      cur += 4 * d * d;
      if ((r = up_f32(&w.b2, d))) return r;
    }
    if ((r = up_f32(&net.lnf_g, d))) return r;
    if ((r = up_f32(&net.lnf_b, d))) return r;
    {   // W_out [d, A] -> fp32 [A, d]
      std::vector<float> tmp(A * d);
      for (size_t i = 0; i < d; ++i)
        for (size_t a = 0; a < A; ++a) tmp[a * d + i] = cur[i * A + a];
      cur += d * A;
      if (dev_alloc(c, net.allocs, &net.W_outT, A * d)) return TSDP_ERR_CUDA;
      CU_TRY(c, cudaMemcpy(net.W_outT, tmp.data(), tmp.size() * sizeof(float), cudaMemcpyHostToDevice));
    }
    if ((r = up_f32(&net.b_out, A))) return r;
    if ((r = up_wT(&net.Wkv_all, wkv_all.data(), d, L * 2 * d))) return r;
    if (dev_alloc(c, net.allocs, &net.bkv_all, L * 2 * d)) return TSDP_ERR_CUDA;
    CU_TRY(c, cudaMemcpy(net.bkv_all, bkv_all.data(), bkv_all.size() * sizeof(float), cudaMemcpyHostToDevice));
    if (dev_alloc(c, net.allocs, &net.kv_time, (size_t)T * L * 2 * d)) return TSDP_ERR_CUDA;
    if (dev_alloc(c, net.allocs, &net.kv_obs, c->items_cap * (To ? To : 1) * L * 2 * d)) return TSDP_ERR_CUDA;
    if ((r = sinus_table((int)d, &net.temb_table))) return r;
    // keys/values of the time token for every timestep: (sinusoidal(tau) + cpos[0]) Wkv2 + bkv2, all blocks
    c->launches_per_round_tmp = 0;
    if (cfg.precision == 0) {
      memtok_kernel<float><<<T, d < 256 ? (int)d : 256>>>(net.temb_table, (int)d, nullptr, nullptr, net.cpos, 0, 0,
                                                           reinterpret_cast<float*>(c->memtok), (int)d);
    } else {
      memtok_kernel<__nv_bfloat16><<<T, d < 256 ? (int)d : 256>>>(net.temb_table, (int)d, nullptr, nullptr, net.cpos, 0, 0,
                                                                   reinterpret_cast<__nv_bfloat16*>(c->memtok), (int)d);
    }
    CU_TRY(c, cudaGetLastError());
    if ((r = gemm(c, c->memtok, net.Wkv_all, net.bkv_all, T, (int)(L * 2 * d), (int)d, EPI_F32, net.kv_time, (int)(L * 2 * d), 0)))
      return r;
    net.fold = xfold_ok(cfg, net.cfg);
    if (net.fold) {
      const size_t per_tok = L * net.cfg.heads * d, rows_obs = c->items_cap * (To ? To : 1);
      std::vector<XfoldLayerW> lw(L);
      for (size_t l = 0; l < L; ++l)
        lw[l] = XfoldLayerW{reinterpret_cast<const __nv_bfloat16*>(net.L[l].Wq2), reinterpret_cast<const __nv_bfloat16*>(net.L[l].Wo2),
                            net.L[l].bq2, net.L[l].ln2_g, net.L[l].ln2_b};
      int st = 0;
      st |= dev_alloc(c, net.allocs, &net.fold_lw, L);
      st |= dev_alloc(c, net.allocs, &net.fold_kq_time, (size_t)T * per_tok);
      st |= dev_alloc(c, net.allocs, &net.fold_ut_time, (size_t)T * per_tok);
      st |= dev_alloc(c, net.allocs, &net.fold_c_time, (size_t)T * L * net.cfg.heads);
      st |= dev_alloc(c, net.allocs, &net.fold_kq_obs, rows_obs * per_tok);
      st |= dev_alloc(c, net.allocs, &net.fold_ut_obs, rows_obs * per_tok);
      st |= dev_alloc(c, net.allocs, &net.fold_c_obs, rows_obs * L * net.cfg.heads);
      if (st) return TSDP_ERR_CUDA;
      CU_TRY(c, cudaMemcpy(net.fold_lw, lw.data(), sizeof(XfoldLayerW) * L, cudaMemcpyHostToDevice));
      if ((r = xfold_build(c, net, net.kv_time, T, net.fold_kq_time, net.fold_ut_time, net.fold_c_time, 0))) return r;
    }
    CU_TRY(c, cudaDeviceSynchronize());
    if ((r = check_status(c))) return r;
  }
  if ((size_t)(cur - blob) != n && net.cfg.arch != TSDP_ARCH_GAUSS) return TSDP_ERR_WEIGHTS;
  net.loaded = true;
  return TSDP_OK;
}

int tsdp_set_schedule(tsdp_ctx* c, const int* Ks, const tsdp_accept_t* accs, int n) {
  if (!c || n < 0 || n > TSDP_MAX_T || (n > 0 && (!Ks || !accs))) return TSDP_ERR_ARG;
  for (int i = 0; i < n; ++i)
    if (Ks[i] < 0 || Ks[i] > c->cfg.max_K || !accept_ok(&accs[i])) return TSDP_ERR_ARG;
  c->sched_K.assign(Ks, Ks + n);
  c->sched_acc.assign(accs, accs + n);
  return TSDP_OK;
}

static int ensure_items(tsdp_ctx* c, size_t N);

int tsdp_request_counts(tsdp_ctx* c, int* h_counts, int n) {
  if (!c || !h_counts || n < 1 || n > c->items_last) return TSDP_ERR_ARG;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  CU_TRY(c, cudaMemcpy(h_counts, c->item_counts, sizeof(int) * 4 * (size_t)n, cudaMemcpyDeviceToHost));
  return TSDP_OK;
}

int tsdp_process_reward(tsdp_ctx* c, float R_final, int T_max, int dt, float* h_reward, int n) {
  if (!c || !h_reward || n < 1 || n > c->items_last || T_max < 1 || dt < 1) return TSDP_ERR_ARG;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  process_reward_kernel<<<(n + 127) / 128, 128>>>(c->item_counts, n, R_final, T_max, dt, c->reward);
  c->launches++;
  CU_TRY(c, cudaGetLastError());
  CU_TRY(c, cudaMemcpy(h_reward, c->reward, sizeof(float) * (size_t)n, cudaMemcpyDeviceToHost));
  return TSDP_OK;
}

int tsdp_set_scheduler(tsdp_ctx* c, int enable) {
  if (!c) return TSDP_ERR_ARG;
  if (enable && !c->sched_loaded) return TSDP_ERR_STATE;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  CU_TRY(c, cudaDeviceSynchronize());
  // captured rounds carry the pointer to the per-environment parameters (or null): capture again
  for (auto& g : c->graphs) cudaGraphExecDestroy(g.second.exec);
  c->graphs.clear();
  c->sched_on = enable != 0;
  return TSDP_OK;
}

int tsdp_set_progress(tsdp_ctx* c, const float* h_progress, int B) {
  if (!c || !h_progress || B < 1) return TSDP_ERR_ARG;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  { int r = ensure_items(c, (size_t)B); if (r) return r; }
  CU_TRY(c, cudaMemcpy(c->progress, h_progress, sizeof(float) * B, cudaMemcpyHostToDevice));
  return TSDP_OK;
}

int tsdp_sched_eval(tsdp_ctx* c, const float* d_obs, const float* d_prev_actions, const float* h_progress, int B,
                    float* h_params, void* stream) {
  if (!c || !d_prev_actions || !h_progress || !h_params || B < 1 || B > c->cfg.max_B) return TSDP_ERR_ARG;
  const int obs_len = c->cfg.obs_tokens * c->cfg.obs_dim;
  if (obs_len > 0 && !d_obs) return TSDP_ERR_ARG;
  if (!c->sched_loaded) return TSDP_ERR_STATE;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  CU_TRY(c, cudaMemcpyAsync(c->progress, h_progress, sizeof(float) * B, cudaMemcpyHostToDevice, s));
  sched_mlp_kernel<<<B, 128, 0, s>>>(c->sched_w, d_obs, obs_len, d_prev_actions, c->D, c->progress, c->cfg.max_K, c->envp,
                                     c->sched_dbg);
  c->launches++;
  CU_TRY(c, cudaGetLastError());
  CU_TRY(c, cudaMemcpyAsync(h_params, c->sched_dbg, sizeof(float) * 8 * B, cudaMemcpyDeviceToHost, s));
  CU_TRY(c, cudaStreamSynchronize(s));
  return TSDP_OK;
}

// Grow the per-request buffers (observations, actions, obs-token K/V, scheduler inputs and outputs) to hold
// N requests.  Captured graphs and tensor maps carry the old addresses, so they are dropped.
static int ensure_items(tsdp_ctx* c, size_t N) {
  if (N <= c->items_cap) return TSDP_OK;
  CU_TRY(c, cudaDeviceSynchronize());
  const tsdp_config_t& cfg = c->cfg;
  const size_t D = c->D, To = cfg.obs_tokens;
  int st = 0;
  st |= dev_alloc(c, c->allocs, &c->actions, N * D);
  st |= dev_alloc(c, c->allocs, &c->obs, N * To * cfg.obs_dim + 1);
  st |= dev_alloc(c, c->allocs, &c->envp, N);
  st |= dev_alloc(c, c->allocs, &c->progress, N);
  st |= dev_alloc(c, c->allocs, &c->sched_dbg, N * 8);
  st |= dev_alloc(c, c->allocs, &c->item_counts, N * 4);
  st |= dev_alloc(c, c->allocs, &c->reward, N);
  size_t dmax = 0;
  for (int w = 0; w < 2; ++w) {
    Net& n = c->net[w];
    if (n.cfg.arch != TSDP_ARCH_XFMR && n.cfg.arch != TSDP_ARCH_DIT) continue;
    dmax = std::max(dmax, (size_t)n.cfg.d);
    if (n.loaded) st |= dev_alloc(c, n.allocs, &n.kv_obs, N * (To ? To : 1) * n.cfg.layers * 2 * n.cfg.d);
    if (n.loaded && n.fold) {
      const size_t rows_obs = N * (To ? To : 1), per_tok = (size_t)n.cfg.layers * n.cfg.heads * n.cfg.d;
      st |= dev_alloc(c, n.allocs, &n.fold_kq_obs, rows_obs * per_tok);
      st |= dev_alloc(c, n.allocs, &n.fold_ut_obs, rows_obs * per_tok);
      st |= dev_alloc(c, n.allocs, &n.fold_c_obs, rows_obs * n.cfg.layers * n.cfg.heads);
    }
  }
  for (int w = 0; w < 2; ++w) {
    Net& n = c->net[w];
    if (n.cfg.arch != TSDP_ARCH_UNET || !n.loaded) continue;
    st |= dev_alloc(c, n.allocs, &n.film_obs, N * n.F);
    st |= dev_alloc(c, n.allocs, &n.obs_m, N * (To * cfg.obs_dim ? To * cfg.obs_dim : 1));
  }
  if (dmax) st |= alloc_bytes(c, c->allocs, &c->memtok, std::max((size_t)cfg.T, N * To) * dmax * (cfg.precision == 0 ? 4 : 2));
  if (st) return TSDP_ERR_CUDA;
  c->items_cap = N;
  for (auto& g : c->graphs) cudaGraphExecDestroy(g.second.exec);
  c->graphs.clear();
  c->maps.clear();
  return TSDP_OK;
}

static int sample_chunk_impl(tsdp_ctx* c, const float* obs, bool obs_on_host, int N, int B, int K, const tsdp_accept_t* acc,
                             uint64_t seed, float* actions, bool actions_on_host, cudaStream_t s) {
  // N requests (environment-chunks) through B slots; N == B is the plain batch
  if (!c || !acc || !actions || B < 1 || B > c->cfg.max_B || N < B || K < 0 || K > c->cfg.max_K || !accept_ok(acc))
    return TSDP_ERR_ARG;
  const size_t obs_n = (size_t)N * c->cfg.obs_tokens * c->cfg.obs_dim;
  if (obs_n > 0 && !obs) return TSDP_ERR_ARG;
  if (!c->net[0].loaded || !c->net[1].loaded) return TSDP_ERR_STATE;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  const int D = c->D, T = c->cfg.T;
  int r;
  if ((r = ensure_items(c, (size_t)N))) return r;
  CU_TRY(c, cudaEventRecord(c->ev_chunk0, s));
  if (obs_n)
    CU_TRY(c, cudaMemcpyAsync(c->obs, obs, obs_n * sizeof(float), obs_on_host ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice, s));
  CU_TRY(c, cudaMemcpyAsync(c->seed, &seed, sizeof(seed), cudaMemcpyHostToDevice, s));
  CU_TRY(c, cudaMemcpyAsync(c->n_items, &N, sizeof(int), cudaMemcpyHostToDevice, s));
  CU_TRY(c, cudaMemsetAsync(c->item_counts, 0, sizeof(int) * 4 * (size_t)N, s));
  c->items_last = N;
  if ((r = upload_schedule(c, K, *acc, s, false))) return r;
  if (c->sched_on) {
    // the scheduler network reads the new observation, the previous chunk's actions and the progress; it
    // runs on a side stream beside the chunk set-up and joins before the first round
    CU_TRY(c, cudaEventRecord(c->ev_fork, s));
    CU_TRY(c, cudaStreamWaitEvent(c->side_stream, c->ev_fork, 0));
    sched_mlp_kernel<<<N, 128, 0, c->side_stream>>>(c->sched_w, c->obs, (int)(obs_n / N), c->actions, D, c->progress,
                                                      c->cfg.max_K, c->envp, nullptr);
    CU_TRY(c, cudaGetLastError());
    CU_TRY(c, cudaEventRecord(c->ev_join, c->side_stream));
    c->launches++;
  }
  const long long xs_b = (long long)(c->cfg.max_K + 1) * D;
  init_chunk_kernel<<<B, 128, 0, s>>>(c->xt, xs_b, c->t, B, D, T, c->seed, c->round_idx, c->n_done, c->item, c->queue_head);
  CU_TRY(c, cudaGetLastError());
  c->launches_per_round_tmp = 0;
  if ((r = prepare_obs(c, c->net[TSDP_BASE], N, s))) return r;
  if ((r = prepare_obs(c, c->net[TSDP_DRAFT], N, s))) return r;
  c->launches += 1 + c->launches_per_round_tmp;
  // Rounds.  A request cannot finish before its drafted windows could have covered T steps, so the
  // completion flag is only read once the slots could have worked through all N requests.
  if (c->sched_on) CU_TRY(c, cudaStreamWaitEvent(s, c->ev_join, 0));
  const int n_sched = (int)c->sched_K.size();
  const long long waves = ((long long)N + B - 1) / B;
  long long budget = (long long)T * N / B;
  const long long max_rounds = (long long)(T + 1) * waves + 1;
  for (long long round = 0; round < max_rounds; ++round) {
    const int Kr = n_sched > 0 ? c->sched_K[round < n_sched ? round : n_sched - 1] : K;
    if ((r = run_round(c, B, Kr, s))) return r;
    c->rounds++;
    budget -= Kr + 1;
    if (budget <= 0) {
      CU_TRY(c, cudaStreamSynchronize(s));
      if (*c->host_done >= N) break;
    }
  }
  CU_TRY(c, cudaMemcpyAsync(actions, c->actions, (size_t)N * D * sizeof(float),
                            actions_on_host ? cudaMemcpyDeviceToHost : cudaMemcpyDeviceToDevice, s));
  CU_TRY(c, cudaEventRecord(c->ev_chunk1, s));
  CU_TRY(c, cudaStreamSynchronize(s));
  {   // device time of this call, copies included, into the latency ring
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->ev_chunk0, c->ev_chunk1) == cudaSuccess) {
      c->lat_ring[c->lat_pos] = ms;
      c->lat_pos = (c->lat_pos + 1) % c->lat_ring.size();
      if (c->lat_n < c->lat_ring.size()) c->lat_n++;
    }
  }
  return check_status(c);
}

int tsdp_sample_chunk(tsdp_ctx* c, const float* d_obs, int B, int K, const tsdp_accept_t* acc, uint64_t seed,
                      float* d_actions, void* stream) {
  return sample_chunk_impl(c, d_obs, false, B, B, K, acc, seed, d_actions, false, reinterpret_cast<cudaStream_t>(stream));
}

int tsdp_serve(tsdp_ctx* c, const float* d_obs, int N, int slots, int K, const tsdp_accept_t* acc, uint64_t seed,
               float* d_actions, void* stream) {
  if (c && slots > N) slots = N;
  return sample_chunk_impl(c, d_obs, false, N, slots, K, acc, seed, d_actions, false, reinterpret_cast<cudaStream_t>(stream));
}

int tsdp_sample_chunk_host(tsdp_ctx* c, const float* h_obs, int B, int K, const tsdp_accept_t* acc, uint64_t seed,
                           float* h_actions) {
  return sample_chunk_impl(c, h_obs, true, B, B, K, acc, seed, h_actions, true, nullptr);
}

int tsdp_round(tsdp_ctx* c, const float* d_obs, int B, int K, const tsdp_accept_t* acc, uint64_t seed, float* d_x,
               int* h_t, float* d_xtilde, float* d_muhat, float* d_eps, float* d_logalpha, int* h_jstar, void* stream) {
  if (!c || !acc || !d_x || !h_t || B < 1 || B > c->cfg.max_B || K < 0 || K > c->cfg.max_K || !accept_ok(acc))
    return TSDP_ERR_ARG;
  for (int b = 0; b < B; ++b)
    if (h_t[b] < -1 || h_t[b] >= c->cfg.T) return TSDP_ERR_ARG;
  const size_t obs_n = (size_t)B * c->cfg.obs_tokens * c->cfg.obs_dim;
  if (obs_n > 0 && !d_obs) return TSDP_ERR_ARG;
  if (!c->net[0].loaded || !c->net[1].loaded) return TSDP_ERR_STATE;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const int D = c->D;
  const size_t K1 = c->cfg.max_K + 1, Km = c->cfg.max_K > 0 ? c->cfg.max_K : 1;
  int r;
  if (obs_n) CU_TRY(c, cudaMemcpyAsync(c->obs, d_obs, obs_n * sizeof(float), cudaMemcpyDeviceToDevice, s));
  CU_TRY(c, cudaMemcpyAsync(c->seed, &seed, sizeof(seed), cudaMemcpyHostToDevice, s));
  if ((r = upload_schedule(c, K, *acc, s, true))) return r;
  CU_TRY(c, cudaMemsetAsync(c->round_idx, 0, sizeof(int), s));
  CU_TRY(c, cudaMemsetAsync(c->n_done, 0, sizeof(int), s));
  {   // every slot serves the request of its own index and nothing is waiting
    std::vector<int> ident(B);
    for (int b = 0; b < B; ++b) ident[b] = b;
    CU_TRY(c, cudaMemcpyAsync(c->item, ident.data(), sizeof(int) * B, cudaMemcpyHostToDevice, s));
    CU_TRY(c, cudaMemcpyAsync(c->queue_head, &B, sizeof(int), cudaMemcpyHostToDevice, s));
    CU_TRY(c, cudaMemcpyAsync(c->n_items, &B, sizeof(int), cudaMemcpyHostToDevice, s));
    CU_TRY(c, cudaMemsetAsync(c->item_counts, 0, sizeof(int) * 4 * (size_t)B, s));
    c->items_last = B;
  }
  CU_TRY(c, cudaMemcpyAsync(c->t, h_t, sizeof(int) * B, cudaMemcpyHostToDevice, s));
  CU_TRY(c, cudaMemcpy2DAsync(c->xt, K1 * D * sizeof(float), d_x, D * sizeof(float), D * sizeof(float), B, cudaMemcpyDeviceToDevice, s));
  c->launches_per_round_tmp = 0;
  if ((r = prepare_obs(c, c->net[TSDP_BASE], B, s))) return r;
  if ((r = prepare_obs(c, c->net[TSDP_DRAFT], B, s))) return r;
  if ((r = enqueue_round(c, B, K, s, true))) return r;
  c->launches += c->launches_per_round_tmp;
  c->cand_static += (uint64_t)B * (K + 1);
  c->rounds++;
  // candidates and drafter means are still intact except slot 0, which now holds the new latent
  if (d_xtilde) {
    CU_TRY(c, cudaMemcpy2DAsync(d_xtilde, (size_t)(K + 1) * D * sizeof(float), c->xt, K1 * D * sizeof(float),
                                (size_t)(K + 1) * D * sizeof(float), B, cudaMemcpyDeviceToDevice, s));
    CU_TRY(c, cudaMemcpy2DAsync(d_xtilde, (size_t)(K + 1) * D * sizeof(float), d_x, D * sizeof(float), D * sizeof(float), B,
                                cudaMemcpyDeviceToDevice, s));
  }
  if (d_muhat && K > 0)
    CU_TRY(c, cudaMemcpy2DAsync(d_muhat, (size_t)K * D * sizeof(float), c->muhat, Km * D * sizeof(float),
                                (size_t)K * D * sizeof(float), B, cudaMemcpyDeviceToDevice, s));
  if (d_eps)
    CU_TRY(c, cudaMemcpy2DAsync(d_eps, (size_t)(K + 1) * D * sizeof(float), c->eps, K1 * D * sizeof(float),
                                (size_t)(K + 1) * D * sizeof(float), B, cudaMemcpyDeviceToDevice, s));
  if (d_logalpha && K > 0)
    CU_TRY(c, cudaMemcpyAsync(d_logalpha, c->dbg_logalpha, sizeof(float) * B * K, cudaMemcpyDeviceToDevice, s));
  CU_TRY(c, cudaMemcpy2DAsync(d_x, D * sizeof(float), c->xt, K1 * D * sizeof(float), D * sizeof(float), B, cudaMemcpyDeviceToDevice, s));
  CU_TRY(c, cudaMemcpyAsync(h_t, c->t, sizeof(int) * B, cudaMemcpyDeviceToHost, s));
  if (h_jstar) CU_TRY(c, cudaMemcpyAsync(h_jstar, c->dbg_jstar, sizeof(int) * B, cudaMemcpyDeviceToHost, s));
  CU_TRY(c, cudaStreamSynchronize(s));
  return check_status(c);
}

int tsdp_denoise(tsdp_ctx* c, int which, const float* d_x, const int* h_tau, const float* d_obs, int N, float* d_eps,
                 void* stream) {
  if (!c || !d_x || !h_tau || !d_eps || N < 1 || N > c->cfg.max_B || (which != TSDP_BASE && which != TSDP_DRAFT))
    return TSDP_ERR_ARG;
  for (int i = 0; i < N; ++i)
    if (h_tau[i] < 0 || h_tau[i] >= c->cfg.T) return TSDP_ERR_ARG;
  const size_t obs_n = (size_t)N * c->cfg.obs_tokens * c->cfg.obs_dim;
  if (obs_n > 0 && !d_obs) return TSDP_ERR_ARG;
  Net& n = c->net[which];
  if (!n.loaded) return TSDP_ERR_STATE;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int r;
  if (obs_n) CU_TRY(c, cudaMemcpyAsync(c->obs, d_obs, obs_n * sizeof(float), cudaMemcpyDeviceToDevice, s));
  CU_TRY(c, cudaMemcpyAsync(c->t, h_tau, sizeof(int) * N, cudaMemcpyHostToDevice, s));
  c->launches_per_round_tmp = 0;
  if ((r = prepare_obs(c, n, N, s))) return r;
  CandMap cm{d_x, (long long)c->D, d_eps, (long long)c->D, c->t, 1, 0, nullptr};
  if ((r = forward(c, n, cm, N, s))) return r;
  c->launches += c->launches_per_round_tmp;
  CU_TRY(c, cudaStreamSynchronize(s));
  return check_status(c);
}

int tsdp_distill_loss(tsdp_ctx* c, const float* d_x0, const float* d_obs, int N, uint64_t seed, float lambda1, float lambda2,
                      double* h_out) {
  if (!c || !d_x0 || !h_out || N < 1 || N > c->cfg.max_B || c->cfg.draft.arch == TSDP_ARCH_FROZEN) return TSDP_ERR_ARG;
  const size_t obs_n = (size_t)N * c->cfg.obs_tokens * c->cfg.obs_dim;
  if (obs_n > 0 && !d_obs) return TSDP_ERR_ARG;
  if (!c->net[0].loaded || !c->net[1].loaded) return TSDP_ERR_STATE;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  cudaStream_t s = nullptr;
  const int D = c->D;
  const long long xs_b = (long long)(c->cfg.max_K + 1) * D;
  int r;
  {   // requests beyond the slots' initial capacity are not involved: sample n uses slot n and request n
    if ((r = ensure_items(c, (size_t)N))) return r;
  }
  if (obs_n) CU_TRY(c, cudaMemcpyAsync(c->obs, d_obs, obs_n * sizeof(float), cudaMemcpyDeviceToDevice, s));
  CU_TRY(c, cudaMemcpyAsync(c->seed, &seed, sizeof(seed), cudaMemcpyHostToDevice, s));
  distill_noise_kernel<<<N, 128, 0, s>>>(c->S, d_x0, c->xt, xs_b, c->t, D, c->seed);
  CU_TRY(c, cudaGetLastError());
  c->launches_per_round_tmp = 1;
  if ((r = prepare_obs(c, c->net[TSDP_BASE], N, s))) return r;
  if ((r = prepare_obs(c, c->net[TSDP_DRAFT], N, s))) return r;
  CandMap cb{c->xt, xs_b, c->eps, xs_b, c->t, 1, 0, nullptr};
  if ((r = forward(c, c->net[TSDP_BASE], cb, N, s))) return r;
  CandMap cd{c->xt, xs_b, c->eps_d, (long long)D, c->t, 1, 0, nullptr};
  if ((r = forward(c, c->net[TSDP_DRAFT], cd, N, s))) return r;
  float* terms = c->muhat;                       // [N, 3] per-sample terms; the drafter means are not in use here
  if ((size_t)3 * N > (size_t)c->cfg.max_B * (c->cfg.max_K > 0 ? c->cfg.max_K : 1) * D) return TSDP_ERR_TOO_LARGE;
  distill_terms_kernel<<<N, 128, 0, s>>>(c->S, c->xt, xs_b, c->eps, xs_b, c->eps_d, (long long)D, c->t, D, terms);
  CU_TRY(c, cudaGetLastError());
  c->launches += c->launches_per_round_tmp + 1;
  std::vector<float> h((size_t)3 * N);
  CU_TRY(c, cudaMemcpyAsync(h.data(), terms, sizeof(float) * 3 * N, cudaMemcpyDeviceToHost, s));
  CU_TRY(c, cudaStreamSynchronize(s));
  if ((r = check_status(c))) return r;
  double sp = 0.0, sn = 0.0, sa = 0.0, cnt = 0.0;
  for (int n = 0; n < N; ++n) {
    sp += h[3 * n];
    if (h[3 * n + 2] > 0.f) { sn += h[3 * n + 1]; sa += erfc(sqrt((double)h[3 * n + 1]) / (2.0 * sqrt(2.0))); cnt += 1.0; }
  }
  h_out[0] = sp / N;
  h_out[1] = cnt > 0 ? sn / cnt : 0.0;
  h_out[2] = (double)lambda1 * h_out[0] + (double)lambda2 * h_out[1];
  h_out[3] = cnt > 0 ? sa / cnt : 1.0;
  return TSDP_OK;
}

int tsdp_distill_step(tsdp_ctx* c, const float* d_x0, const float* d_obs, int N, uint64_t seed, float lambda1, float lambda2,
                      float lr, double* h_out) {
  if (!c || !d_x0 || !h_out || N < 1 || N > c->cfg.max_B || c->cfg.draft.arch != TSDP_ARCH_GAUSS || c->cfg.clip > 0.f ||
      !(lr >= 0.f))
    return TSDP_ERR_ARG;
  const size_t obs_n = (size_t)N * c->cfg.obs_tokens * c->cfg.obs_dim;
  if (obs_n > 0 && !d_obs) return TSDP_ERR_ARG;
  if (!c->net[0].loaded || !c->net[1].loaded) return TSDP_ERR_STATE;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  cudaStream_t s = nullptr;
  const int D = c->D;
  const long long xs_b = (long long)(c->cfg.max_K + 1) * D;
  Net& dn = c->net[TSDP_DRAFT];
  int r;
  if ((r = ensure_items(c, (size_t)N))) return r;
  if (obs_n) CU_TRY(c, cudaMemcpyAsync(c->obs, d_obs, obs_n * sizeof(float), cudaMemcpyDeviceToDevice, s));
  CU_TRY(c, cudaMemcpyAsync(c->seed, &seed, sizeof(seed), cudaMemcpyHostToDevice, s));
  const float theta[2] = {dn.m0, dn.s0};
  CU_TRY(c, cudaMemcpyAsync(c->distill_theta, theta, sizeof(theta), cudaMemcpyHostToDevice, s));
  distill_noise_kernel<<<N, 128, 0, s>>>(c->S, d_x0, c->xt, xs_b, c->t, D, c->seed);
  CU_TRY(c, cudaGetLastError());
  c->launches_per_round_tmp = 1;
  if ((r = prepare_obs(c, c->net[TSDP_BASE], N, s))) return r;
  CandMap cb{c->xt, xs_b, c->eps, xs_b, c->t, 1, 0, nullptr};
  if ((r = forward(c, c->net[TSDP_BASE], cb, N, s))) return r;
  distill_gauss_grad_kernel<<<N, 128, 0, s>>>(c->S, c->xt, xs_b, c->eps, xs_b, c->t, D, c->distill_theta, c->distill_terms);
  distill_gauss_update_kernel<<<1, 256, 0, s>>>(c->distill_terms, N, lambda1, lambda2, lr, c->distill_theta, c->distill_res);
  CU_TRY(c, cudaGetLastError());
  c->launches += c->launches_per_round_tmp + 2;
  CU_TRY(c, cudaMemcpyAsync(h_out, c->distill_res, sizeof(double) * 7, cudaMemcpyDeviceToHost, s));
  CU_TRY(c, cudaStreamSynchronize(s));
  if ((r = check_status(c))) return r;
  // the drafter's parameters travel to its kernels by value: adopt the new ones and drop rounds captured with the old
  dn.m0 = (float)h_out[5];
  dn.s0 = (float)h_out[6];
  for (auto& g : c->graphs) cudaGraphExecDestroy(g.second.exec);
  c->graphs.clear();
  return TSDP_OK;
}

int tsdp_gemm(tsdp_ctx* c, const void* d_A, const void* d_W, const float* d_bias, int M, int N, int K, int epi,
              void* d_out, void* stream) {
  if (!c || !d_A || !d_W || !d_out || M < 1 || N < 1 || K < 1 || epi < 0 || epi > 4) return TSDP_ERR_ARG;
  if (epi == 4 && (c->cfg.precision != 1 || N != 3 * K || K % 64 != 0 || M % 16 != 0)) return TSDP_ERR_ARG;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (c->cfg.precision == 0 && epi == EPI_STORE) epi = EPI_F32;
  c->launches_per_round_tmp = 0;
  c->dbg_in_test_gemm = true;
  int r = epi == 4 ? gemm_qkv_attn_raw(c, d_A, d_W, d_bias, M, K, d_out, s) : gemm(c, d_A, d_W, d_bias, M, N, K, epi, d_out, N, s);
  c->dbg_in_test_gemm = false;
  c->launches += c->launches_per_round_tmp;
  if (r) return r;
  CU_TRY(c, cudaStreamSynchronize(s));
  // test interface: operands are caller-owned and may be freed, so their tensor maps are not kept
  c->maps.clear();
  return check_status(c);
}

int tsdp_debug_check_guards(tsdp_ctx* c, int* h_checked) {
  if (!c) return TSDP_ERR_ARG;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  CU_TRY(c, cudaDeviceSynchronize());
  uint8_t tail[GUARD_BYTES];
  int n = 0;
  for (const auto& g : c->guards) {
    CU_TRY(c, cudaMemcpy(tail, static_cast<const uint8_t*>(g.first) + g.second, GUARD_BYTES, cudaMemcpyDeviceToHost));
    for (size_t i = 0; i < GUARD_BYTES; ++i)
      if (tail[i] != GUARD_PATTERN) {
        c->last_error = "guard bytes behind a device buffer of " + std::to_string(g.second) + " bytes were overwritten (offset " +
                        std::to_string(i) + ")";
        if (h_checked) *h_checked = n;
        return TSDP_ERR_OVERRUN;
      }
    ++n;
  }
  if (h_checked) *h_checked = n;
  return TSDP_OK;
}

int tsdp_debug_arm_gemm_timeout(tsdp_ctx* c, long long wait_cycles) {
  if (!c || wait_cycles < 1000 || wait_cycles > 2000000000ll || c->cfg.precision != 1) return TSDP_ERR_ARG;
  c->dbg_armed = true;
  c->dbg_wait_cycles = wait_cycles;
  return TSDP_OK;
}

int tsdp_gemm_timed(tsdp_ctx* c, const void* d_A, const void* d_W, const float* d_bias, int M, int N, int K, int epi,
                    void* d_out, int reps, float* h_ms, void* stream) {
  if (!c || !d_A || !d_W || !d_out || !h_ms || M < 1 || N < 1 || K < 1 || epi < 0 || epi > 4 || reps < 1)
    return TSDP_ERR_ARG;
  if (epi == 4 && (c->cfg.precision != 1 || N != 3 * K || K % 64 != 0 || M % 16 != 0)) return TSDP_ERR_ARG;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  cudaStream_t s_ = s;
  if (c->cfg.precision == 0 && epi == EPI_STORE) epi = EPI_F32;
  auto one = [&]() {
    return epi == 4 ? gemm_qkv_attn_raw(c, d_A, d_W, d_bias, M, K, d_out, s_) : gemm(c, d_A, d_W, d_bias, M, N, K, epi, d_out, N, s_);
  };
  cudaEvent_t e0, e1;
  CU_TRY(c, cudaEventCreate(&e0));
  CU_TRY(c, cudaEventCreate(&e1));
  c->launches_per_round_tmp = 0;
  int r = one();     // builds the tensor maps, warms up
  cudaEventRecord(e0, s);
  for (int i = 0; i < reps && r == TSDP_OK; ++i) r = one();
  cudaEventRecord(e1, s);
  c->launches += c->launches_per_round_tmp;
  cudaError_t e = cudaStreamSynchronize(s);
  float ms = 0.f;
  if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  c->maps.clear();
  if (r) return r;
  CU_TRY(c, e);
  *h_ms = ms / reps;
  return check_status(c);
}

int tsdp_stats(tsdp_ctx* c, tsdp_stats_t* out) {
  if (!c || !out) return TSDP_ERR_ARG;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  CU_TRY(c, cudaDeviceSynchronize());
  std::vector<DevStats> staging(1);
  DevStats& ds = staging[0];
  CU_TRY(c, cudaMemcpy(&ds, c->stats, sizeof(DevStats), cudaMemcpyDeviceToHost));
  memset(out, 0, sizeof(*out));
  out->chunks = ds.chunks_done;
  out->rounds = c->rounds;
  out->env_rounds = ds.env_rounds;
  out->base_evals = ds.base_evals;
  out->draft_evals = ds.draft_evals;
  out->drafts_tested = ds.drafts_tested;
  out->drafts_accepted = ds.drafts_accepted;
  out->rejections = ds.rejections;
  out->bonus_steps = ds.bonus_steps;
  out->steps_advanced = ds.steps_advanced;
  out->draft_rounds = ds.draft_rounds;
  out->cand_dense = c->cand_static;
  out->cand_computed = ds.cand_computed > 0 || c->compact ? ds.cand_computed : c->cand_static;
  out->nfe = (double)ds.env_rounds + (double)c->cfg.draft_nfe * (double)ds.draft_evals;
  if (c->cfg.draft.arch == TSDP_ARCH_FROZEN) out->nfe = (double)ds.env_rounds + (double)ds.draft_rounds;
  out->call_ms_samples = c->lat_n;
  if (c->lat_n > 0) {   // nearest-rank percentiles over the ring
    std::vector<float> v(c->lat_ring.begin(), c->lat_ring.begin() + c->lat_n);
    std::sort(v.begin(), v.end());
    auto pct = [&](double q) { size_t i = (size_t)std::ceil(q * v.size()); return (double)v[i > 0 ? i - 1 : 0]; };
    out->call_ms_p50 = pct(0.50);
    out->call_ms_p99 = pct(0.99);
  }
  for (int i = 0; i < TSDP_MAX_T; ++i) {
    out->hist_drafted[i] = ds.hist_drafted[i];
    out->hist_tested[i] = ds.hist_tested[i];
    out->hist_accepted[i] = ds.hist_accepted[i];
  }
  return TSDP_OK;
}

int tsdp_reset_stats(tsdp_ctx* c) {
  if (!c) return TSDP_ERR_ARG;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  CU_TRY(c, cudaDeviceSynchronize());
  CU_TRY(c, cudaMemset(c->stats, 0, sizeof(DevStats)));
  c->rounds = 0;
  c->launches = 0;
  c->cand_static = 0;
  c->lat_pos = c->lat_n = 0;
  return TSDP_OK;
}

uint64_t tsdp_kernel_launches(const tsdp_ctx* c) { return c ? c->launches : 0; }

int tsdp_profile(tsdp_ctx* c, int enable) {
  if (!c) return TSDP_ERR_ARG;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  CU_TRY(c, cudaDeviceSynchronize());
  for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
  c->prof_ev.clear(); c->prof_cat.clear(); c->prof_flop.clear();
  c->prof_on = enable != 0;
  return TSDP_OK;
}

int tsdp_profile_read(tsdp_ctx* c, double* ms, double* flop, uint64_t* launches) {
  if (!c || !ms || !flop || !launches) return TSDP_ERR_ARG;
  CU_TRY(c, cudaSetDevice(c->cfg.device));
  CU_TRY(c, cudaDeviceSynchronize());
  for (int i = 0; i < TSDP_PROF_FAMILIES; ++i) { ms[i] = 0.0; flop[i] = 0.0; launches[i] = 0; }
  for (size_t i = 0; i < c->prof_cat.size(); ++i) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]) != cudaSuccess) continue;
    const int k = c->prof_cat[i];
    ms[k] += t; flop[k] += c->prof_flop[i]; launches[k] += 1;
  }
  return TSDP_OK;
}


// ------------------------------------------------------------------------------------------------
// Allocation-free verification tail.
//
// The working memory of this entry point is a file-scope device array: it is part of the library
// image on every GPU that loads it and lives until the process exits.  Host code never passes the
// array's name to a kernel (on the host that name is only a stand-in); its device address is looked
// up once per device with cudaGetSymbolAddress and kept in g_static_addr.
// ------------------------------------------------------------------------------------------------
namespace {
constexpr size_t ST_OFF_STATS = 0;                                            // DevStats
constexpr size_t ST_OFF_TAB = 24832;                                          // 5 x TSDP_STATIC_MAX_T floats
constexpr size_t ST_OFF_T = ST_OFF_TAB + 5 * TSDP_STATIC_MAX_T * 4;           // t[B]
constexpr size_t ST_OFF_J = ST_OFF_T + TSDP_STATIC_MAX_B * 4;                 // j*[B]
constexpr size_t ST_OFF_MISC = ST_OFF_J + TSDP_STATIC_MAX_B * 4;              // seed, round index, done count, round parameters
constexpr size_t ST_BYTES = ST_OFF_MISC + 256;
static_assert(sizeof(DevStats) <= ST_OFF_TAB, "statistics block overlaps the tables");
static_assert(ST_OFF_TAB % 256 == 0 && ST_OFF_T % 256 == 0 && ST_OFF_J % 256 == 0 && ST_OFF_MISC % 256 == 0, "alignment");
static_assert(ST_BYTES <= 64 * 1024, "static scratch is meant to stay small");
}  // namespace

static __device__ __align__(256) unsigned char g_static_scratch[ST_BYTES];

namespace {
constexpr int ST_MAX_DEVICES = 64;
unsigned char* g_static_addr[ST_MAX_DEVICES] = {};
}  // namespace

int tsdp_verify_commit_static(int device, int T, float beta0, float beta1, float clip, float* d_xt,
                              const float* d_muhat, const float* d_eps, const int* h_t, int B, int K, int D,
                              const tsdp_accept_t* acc, uint64_t seed, float draft_nfe, float* d_actions,
                              int* h_t_new, int* h_jstar, float* d_logalpha, void* stream) {
  if (!d_xt || !d_eps || !h_t || !acc || !d_actions || !h_t_new || !h_jstar || (K > 0 && !d_muhat) || B < 1 || K < 0 ||
      D < 1 || T < 1 || device < 0 || device >= ST_MAX_DEVICES || !(beta0 > 0.f) || !(beta1 < 1.f) || !accept_ok(acc))
    return TSDP_ERR_ARG;
  if (B > TSDP_STATIC_MAX_B || T > TSDP_STATIC_MAX_T || K > TSDP_MAX_K) {
    fprintf(stderr, "tsdp_verify_commit_static: B = %d, T = %d, K = %d exceed the built-in capacity (B <= %d, T <= %d, K <= %d)\n",
            B, T, K, (int)TSDP_STATIC_MAX_B, (int)TSDP_STATIC_MAX_T, (int)TSDP_MAX_K);
    return TSDP_ERR_TOO_LARGE;
  }
  for (int b = 0; b < B; ++b)
    if (h_t[b] < -1 || h_t[b] >= T) return TSDP_ERR_ARG;
#define ST_TRY(expr)                                                                              \
  do {                                                                                            \
    cudaError_t e__ = (expr);                                                                     \
    if (e__ != cudaSuccess) {                                                                     \
      fprintf(stderr, "tsdp_verify_commit_static: %s: %s\n", #expr, cudaGetErrorString(e__));    \
      return TSDP_ERR_CUDA;                                                                       \
    }                                                                                             \
  } while (0)
  ST_TRY(cudaSetDevice(device));
  if (!g_static_addr[device]) {   // first call on this device: resolve the array's device address
    void* p = nullptr;
    ST_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
    g_static_addr[device] = reinterpret_cast<unsigned char*>(p);
  }
  unsigned char* base = g_static_addr[device];
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  DevStats* st = reinterpret_cast<DevStats*>(base + ST_OFF_STATS);
  float* dtab = reinterpret_cast<float*>(base + ST_OFF_TAB);
  int* dt = reinterpret_cast<int*>(base + ST_OFF_T);
  int* dj = reinterpret_cast<int*>(base + ST_OFF_J);
  uint64_t* dseed = reinterpret_cast<uint64_t*>(base + ST_OFF_MISC);
  int* dround = reinterpret_cast<int*>(base + ST_OFF_MISC + 8);
  int* ddone = reinterpret_cast<int*>(base + ST_OFF_MISC + 12);
  RoundParams* drp = reinterpret_cast<RoundParams*>(base + ST_OFF_MISC + 16);

  float tab[5 * TSDP_STATIC_MAX_T];
  {
    double abar = 1.0, abar_prev = 1.0;
    for (int t = 0; t < T; ++t) {
      const double beta = T > 1 ? beta0 + ((double)beta1 - beta0) * t / (T - 1) : beta0;
      const double alpha = 1.0 - beta;
      abar_prev = abar;
      abar *= alpha;
      tab[0 * T + t] = (float)std::sqrt(abar);
      tab[1 * T + t] = (float)std::sqrt(1.0 - abar);
      tab[2 * T + t] = (float)(std::sqrt(abar_prev) * beta / (1.0 - abar));
      tab[3 * T + t] = (float)(std::sqrt(alpha) * (1.0 - abar_prev) / (1.0 - abar));
      tab[4 * T + t] = (float)std::sqrt(beta * (1.0 - abar_prev) / (1.0 - abar));
    }
  }
  RoundParams rp;
  fill_round_params(&rp, K, *acc);
  // the array keeps whatever the previous call left: counters and indices start from zero again
  ST_TRY(cudaMemsetAsync(base + ST_OFF_STATS, 0, sizeof(DevStats), s));
  ST_TRY(cudaMemsetAsync(base + ST_OFF_MISC, 0, 256, s));
  ST_TRY(cudaMemcpyAsync(dtab, tab, sizeof(float) * 5 * T, cudaMemcpyHostToDevice, s));
  ST_TRY(cudaMemcpyAsync(dt, h_t, sizeof(int) * B, cudaMemcpyHostToDevice, s));
  ST_TRY(cudaMemcpyAsync(dseed, &seed, sizeof(seed), cudaMemcpyHostToDevice, s));
  ST_TRY(cudaMemcpyAsync(drp, &rp, sizeof(rp), cudaMemcpyHostToDevice, s));
  const DdpmTables S{dtab, dtab + T, dtab + 2 * T, dtab + 3 * T, dtab + 4 * T, T, clip};
  const long long xs_b = (long long)(K + 1) * D, ms_b = (long long)(K > 0 ? K : 1) * D;
  int warps = K < 1 ? 1 : K;
  if (warps < 4) warps = 4;
  if (warps > 16) warps = 16;
  accept_kernel<<<B, warps * 32, 0, s>>>(S, d_xt, xs_b, d_muhat, ms_b, d_eps, xs_b, dt, K, D, dseed, drp, 1, dround,
                                         d_actions, ddone, st, draft_nfe, d_logalpha, dj, nullptr, nullptr, nullptr, nullptr, nullptr);
  ST_TRY(cudaGetLastError());
  ST_TRY(cudaMemcpyAsync(h_t_new, dt, sizeof(int) * B, cudaMemcpyDeviceToHost, s));
  ST_TRY(cudaMemcpyAsync(h_jstar, dj, sizeof(int) * B, cudaMemcpyDeviceToHost, s));
  ST_TRY(cudaStreamSynchronize(s));
#undef ST_TRY
  return TSDP_OK;
}

}  // extern "C"
