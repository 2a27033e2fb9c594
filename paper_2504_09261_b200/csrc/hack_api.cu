// Host side of the C ABI: argument checks, the per-layer state machine, the deterministic length
// plan of every step, cache and scratch allocation, and the launch sequence of the step.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <utility>

#include "hack_internal.h"

namespace hack {

static thread_local std::string g_last_error;
void set_error(const std::string& msg) { g_last_error = msg; }

bool allow_dynamic_smem_impl(const void* kern, size_t bytes) {
  static std::mutex mu;
  static std::vector<std::pair<const void*, int>> done;        // (kernel, device) pairs already served
  int dev = 0;
  cudaGetDevice(&dev);
  std::lock_guard<std::mutex> lock(mu);
  for (const auto& kd : done)
    if (kd.first == kern && kd.second == dev) return true;
  const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e != cudaSuccess) {
    set_error(std::string("cudaFuncSetAttribute(MaxDynamicSharedMemorySize): ") + cudaGetErrorString(e));
    return false;
  }
  done.emplace_back(kern, dev);
  return true;
}

int sm_count() {
  static std::mutex mu;
  static int count[64] = {0};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return 148;
  std::lock_guard<std::mutex> lock(mu);
  if (count[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
    count[dev] = n;
  }
  return count[dev];
}

bool attend_tc_serves(const StepArgs& a, int dtype) {
  // the tensor-core kernel serves bf16 caches once a scale has enough rows for its TMA boxes
  return dtype == HACK_BF16 && a.k_map && a.n_new >= kTcMinQueries && (long long)a.batch * a.n_heads * a.n_new >= 128;
}

int launch_attend(const StepArgs& a, int dtype, const void* q, void* out, cudaStream_t st) {
  if (attend_tc_serves(a, dtype))
    return launch_attend_tc(a, a.k_map, a.v_map, a.head_order, q, out, nullptr, nullptr, nullptr, 0, false, st);
  return launch_attend_simt(a, dtype, q, out, st);
}

}  // namespace hack

using hack::set_error;

struct LayerState {
  int next_scale = 0;
  int phase = 0;          // 0: scale not started; 1: compacted, attention pending
  int len[2] = {0, 0};    // stored length per head type ([0] structural, [1] contextual)
};

struct alignas(64) TensorMapBox { unsigned char bytes[128]; };

#if defined(HACK_DEBUG_CHECKS)
constexpr int kCanaryRows = 1;
#else
constexpr int kCanaryRows = 0;
#endif

struct hack_cache {
  hack_config_t cfg;
  std::vector<int32_t> sides, n_tok, t_cum;     // t_cum[k] = tokens of scales 0..k
  std::vector<uint8_t> mask;                    // host copy [L*H]
  int elt = 2;
  int budget[2] = {0, 0};
  int cap[2] = {0, 0};
  int t_init = 0;
  float sm_scale = 0.f;
  hack_limits_t limits{};
  std::vector<LayerState> layers;
  std::vector<size_t> layer_rows;               // rows per plane of each layer
  std::vector<size_t> layer_row_base;           // first row of each layer inside the big planes
  std::vector<int> n_ctx_heads;                 // contextual heads per layer
  // device memory
  unsigned char* k_all = nullptr;
  unsigned char* v_all = nullptr;
  int32_t* pos_all = nullptr;
  int32_t* row_off = nullptr;                   // [L][b*H]
  std::vector<int32_t> row_off_host;            // same table on the host
  uint8_t* mask_dev = nullptr;                  // [L*H]
  float* scores = nullptr;                      // [b*H, cand_stride]
  int32_t* idx = nullptr;                       // [b*H, kept_stride]
  hack::Scratch scratch{};
  int* status = nullptr;
  int32_t* n_old = nullptr;                     // [b*H] scratch of the compaction kernels
  hack::MergeScratch merge{};                   // merge_last: scratch of the final-scale merge
  TensorMapBox merge_ev_map;
  float* attn_row_stats = nullptr;              // bf16 caches: [b*H, max N_k, 2] softmax row statistics (Eq. 6 path)
  float* attn_block_var = nullptr;              // bf16 caches: [b*H, var_blocks] per key block variances
  int var_blocks = 0;
  int32_t* obs_rows = nullptr;                  // HACK_OBS_CALLER: [n_scales][kMaxObs] query rows of Q~
  std::vector<uint8_t> obs_rows_set;            // per scale: rows were supplied
  std::vector<TensorMapBox> k_maps, v_maps;     // per layer, bf16 caches only
  int32_t* head_order = nullptr;                // [L][2][b*H]: [0] structural heads first, [1] contextual first
  // host-buffer entry point: kHostSlots staging sets (q, k, v, o) cycled call by call, copies on
  // two private streams so that the next call's upload runs under this call's kernels
  static constexpr int kHostSlots = 3;
  unsigned char* stage[kHostSlots][4] = {};
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  cudaEvent_t ev_in[kHostSlots] = {}, ev_step[kHostSlots] = {}, ev_out[kHostSlots] = {};
  uint64_t host_calls = 0;
  size_t reserved_bytes = 0, peak_bytes = 0;
  uint64_t launches = 0;
  long long wait_cycles = hack::kDefaultWaitCycles;   // limit of the kernels' bounded waits
  // fused step with one head type compressing: the attention of the other type runs beside the
  // compression on this stream, forked from and joined to the caller's stream by the two events
  cudaStream_t side_stream = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  bool poisoned = false;                        // a launch failed after part of a step had been enqueued
  // optional per-stage device timing (score, select, compact, attend)
  bool timing = false;
  std::vector<cudaEvent_t> ev_pool;
  size_t ev_used = 0;
  struct Span { int stage; size_t e0, e1; int launches; };
  std::vector<Span> spans;
  double stage_ms[4] = {0, 0, 0, 0};
  uint64_t stage_launches[4] = {0, 0, 0, 0};
};

namespace {

#define HACK_CUDA(call)                                                              \
  do {                                                                               \
    cudaError_t e_ = (call);                                                         \
    if (e_ != cudaSuccess) {                                                         \
      set_error(std::string(#call) + ": " + cudaGetErrorString(e_));                 \
      return e_ == cudaErrorMemoryAllocation ? HACK_ERR_OOM : HACK_ERR_CUDA;         \
    }                                                                                \
  } while (0)

hack_status_t fail(hack_status_t s, const char* msg) {
  set_error(msg);
  return s;
}

// Length plan of one step from the layer's current lengths.  Pure host arithmetic: the stored
// length after a step depends on the schedule, the budget and the head type only.
void plan_step(const hack_cache* c, const LayerState& ls, int scale, hack_step_info_t* p) {
  const int n_new = c->n_tok[scale];
  p->n_new = n_new;
  p->n_obs_rows = std::min(c->cfg.n_obs, n_new);
  int cand[2], kept[2], trig[2];
  for (int t = 0; t < 2; ++t) {
    const int L = ls.len[t];
    cand[t] = L + n_new;
    if (cand[t] <= c->budget[t]) {            // compress only when the budget is exceeded
      kept[t] = cand[t];
      trig[t] = 0;
    } else {
      trig[t] = 1;
      if (t == 1) {
        kept[t] = c->budget[t];
      } else {
        int prot;
        if (scale < c->cfg.n_init_scales) prot = cand[t];
        else if (c->cfg.overflow_policy == HACK_OVERFLOW_KEEP_PROTECTED) prot = std::min(L, c->t_init) + n_new;
        else prot = std::min(L, c->t_init);
        kept[t] = std::min(cand[t], std::max(c->budget[t], prot));
      }
    }
  }
  p->stored_s = ls.len[0]; p->stored_c = ls.len[1];
  p->cand_s = cand[0];     p->cand_c = cand[1];
  p->kept_s = kept[0];     p->kept_c = kept[1];
  p->triggered_s = trig[0]; p->triggered_c = trig[1];
}

hack::StepArgs make_args(const hack_cache* c, int layer, int scale, const hack_step_info_t& p) {
  hack::StepArgs a{};
  a.n_heads = c->cfg.n_heads; a.batch = c->cfg.batch; a.head_dim = c->cfg.head_dim;
  a.n_new = p.n_new;
  a.stored[0] = p.stored_s; a.stored[1] = p.stored_c;
  a.cand[0] = p.cand_s;     a.cand[1] = p.cand_c;
  a.kept[0] = p.kept_s;     a.kept[1] = p.kept_c;
  a.cap[0] = c->cap[0];     a.cap[1] = c->cap[1];
  a.trig[0] = p.triggered_s; a.trig[1] = p.triggered_c;
  a.n_obs_rows = p.n_obs_rows;
  // the query subset of Eq. 9: uniform spacing, or one of the ablation's alternatives
  a.obs_first = c->cfg.obs_sampler == HACK_OBS_RECENT ? p.n_new - p.n_obs_rows : 0;
  a.obs_span = c->cfg.obs_sampler == HACK_OBS_UNIFORM ? p.n_new : p.n_obs_rows;
  a.obs_rows = c->cfg.obs_sampler == HACK_OBS_CALLER ? c->obs_rows + (size_t)scale * hack::kMaxObs : nullptr;
  a.obs_full = c->cfg.obs_sampler == HACK_OBS_FULL;
  a.sm_scale = c->sm_scale;
  a.wait_cycles = c->wait_cycles;
  a.t_init = c->t_init;
  a.protect_new = (c->cfg.overflow_policy == HACK_OVERFLOW_KEEP_PROTECTED) || scale < c->cfg.n_init_scales;
  a.pos_base = scale == 0 ? 0 : c->t_cum[scale - 1];
  a.cand_stride = c->limits.cand_stride;
  a.kept_stride = c->limits.kept_stride;
  a.is_ctx = c->mask_dev + (size_t)layer * c->cfg.n_heads;
  a.row_off = c->row_off + (size_t)layer * c->cfg.batch * c->cfg.n_heads;
  const size_t row_bytes = (size_t)c->cfg.head_dim * c->elt;
  a.k_plane = c->k_all + c->layer_row_base[layer] * row_bytes;
  a.v_plane = c->v_all + c->layer_row_base[layer] * row_bytes;
  a.pos_plane = c->pos_all + c->layer_row_base[layer];
  a.status = c->status;
  a.n_old = c->n_old;
  if (!c->k_maps.empty()) {
    a.k_map = &c->k_maps[layer];
    a.v_map = &c->v_maps[layer];
    const int bh = c->cfg.batch * c->cfg.n_heads;
    a.head_order = c->head_order + ((size_t)layer * 2 + (p.kept_c > p.kept_s ? 1 : 0)) * bh;
  }
  return a;
}

size_t live_bytes(const hack_cache* c) {
  size_t rows = 0;
  for (int l = 0; l < c->cfg.n_layers; ++l) {
    const LayerState& ls = c->layers[l];
    rows += (size_t)c->cfg.batch * ((size_t)c->n_ctx_heads[l] * ls.len[1] +
                                    (size_t)(c->cfg.n_heads - c->n_ctx_heads[l]) * ls.len[0]);
  }
  return rows * c->cfg.head_dim * c->elt * 2;
}

// Makes the cache's device current for the duration of an entry point and puts the caller's back.
struct DeviceScope {
  int prev = -1;
  bool switched = false;
  cudaError_t err = cudaSuccess;
  explicit DeviceScope(int want) {
    err = cudaGetDevice(&prev);
    if (err == cudaSuccess && prev != want) {
      err = cudaSetDevice(want);
      switched = err == cudaSuccess;
    }
  }
  ~DeviceScope() { if (switched) cudaSetDevice(prev); }
};
#define HACK_ON_DEVICE(c)                                                                        \
  DeviceScope dev_scope_((c)->cfg.device);                                                       \
  if (dev_scope_.err != cudaSuccess) {                                                           \
    set_error(std::string("selecting the cache's device: ") + cudaGetErrorString(dev_scope_.err)); \
    return HACK_ERR_CUDA;                                                                        \
  }

// A launcher failed after earlier launches of the same step were enqueued: the device-side state
// of the layer no longer matches the host's plan, so the cache refuses further steps until reset.
hack_status_t poison(hack_cache* c) {
  c->poisoned = true;
  return HACK_ERR_CUDA;   // text recorded by the launcher
}

hack_status_t check_step(const hack_cache* c, int layer, int scale, int want_phase) {
  if (!c) return fail(HACK_ERR_INVALID_ARG, "cache is NULL");
  if (c->poisoned)
    return fail(HACK_ERR_STATE, "an earlier step failed half way (a kernel launch was refused); call hack_reset before the next image");
  if (layer < 0 || layer >= c->cfg.n_layers) return fail(HACK_ERR_INVALID_ARG, "layer out of range");
  if (scale < 0 || scale >= c->cfg.n_scales) return fail(HACK_ERR_INVALID_ARG, "scale out of range");
  const LayerState& ls = c->layers[layer];
  if (scale != ls.next_scale) return fail(HACK_ERR_STATE, "this layer expects a different scale");
  if (ls.phase != want_phase)
    return fail(HACK_ERR_STATE, want_phase ? "hack_compact must precede hack_attend for this scale"
                                           : "this scale is already compacted; call hack_attend");
  return HACK_OK;
}

// Brackets one stage's launches with two events when stage timing is on.
struct StageScope {
  hack_cache* c; cudaStream_t st; int stage; size_t e0 = 0; bool on;
  StageScope(hack_cache* c_, cudaStream_t st_, int stage_) : c(c_), st(st_), stage(stage_), on(c_->timing) {
    if (!on) return;
    e0 = grab();
    cudaEventRecord(c->ev_pool[e0], st);
  }
  size_t grab() {
    if (c->ev_used == c->ev_pool.size()) {
      cudaEvent_t e;
      cudaEventCreate(&e);
      c->ev_pool.push_back(e);
    }
    return c->ev_used++;
  }
  void done(int launches) {
    if (!on) return;
    const size_t e1 = grab();
    cudaEventRecord(c->ev_pool[e1], st);
    c->spans.push_back({stage, e0, e1, launches});
  }
};

bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

void advance_after_compact(hack_cache* c, int layer, const hack_step_info_t& p) {
  LayerState& ls = c->layers[layer];
  ls.len[0] = p.kept_s;
  ls.len[1] = p.kept_c;
  ls.phase = 1;
  c->peak_bytes = std::max(c->peak_bytes, live_bytes(c));
}

}  // namespace

extern "C" {

const char* hack_last_error(void) { return hack::g_last_error.c_str(); }

hack_status_t hack_split_budget(int32_t budget, double alpha, int32_t rule, double param,
                                int32_t total_tokens, int32_t* budget_c, int32_t* budget_s) {
  if (!budget_c || !budget_s) return fail(HACK_ERR_INVALID_ARG, "output pointer is NULL");
  if (!(alpha > 0.0 && alpha < 1.0)) return fail(HACK_ERR_INVALID_ARG, "alpha must be in (0,1)");
  if (budget < 1 || total_tokens < 1 || !(param > 0.0)) return fail(HACK_ERR_INVALID_ARG, "budget, total_tokens and param must be positive");
  const double eps = 1e-9;
  long long bc, bs;
  if (rule == 0) {
    bc = (long long)std::floor(param * total_tokens + eps);
    bs = (long long)std::floor((budget - alpha * (double)bc) / (1.0 - alpha) + eps);
  } else if (rule == 1) {
    bc = (long long)std::floor(budget / (alpha + param * (1.0 - alpha)) + eps);
    bs = (long long)std::llround(param * (double)bc);
  } else {
    return fail(HACK_ERR_INVALID_ARG, "rule must be 0 (fraction) or 1 (ratio)");
  }
  bs = std::min<long long>(bs, total_tokens);
  *budget_c = (int32_t)std::max<long long>(bc, 1);
  *budget_s = (int32_t)std::max<long long>(bs, 1);
  return HACK_OK;
}

hack_status_t hack_init_cache(const hack_config_t* cfg, hack_cache_t** out) {
  if (!cfg || !out) return fail(HACK_ERR_INVALID_ARG, "cfg or out is NULL");
  if (!cfg->scale_sides || !cfg->head_is_contextual) return fail(HACK_ERR_INVALID_ARG, "scale_sides or head_is_contextual is NULL");
  if (cfg->n_layers < 1 || cfg->n_heads < 1 || cfg->batch < 1 || cfg->n_scales < 1)
    return fail(HACK_ERR_INVALID_ARG, "n_layers, n_heads, batch and n_scales must be positive");
  if (cfg->budget_c < 1 || cfg->budget_s < 1) return fail(HACK_ERR_INVALID_ARG, "budgets must be at least 1");
  if (cfg->n_init_scales < 0 || cfg->n_init_scales > cfg->n_scales) return fail(HACK_ERR_INVALID_ARG, "n_init_scales out of range");
  if (cfg->overflow_policy != 0 && cfg->overflow_policy != 1) return fail(HACK_ERR_INVALID_ARG, "unknown overflow_policy");
  if (cfg->sm_scale < 0.f || !std::isfinite(cfg->sm_scale)) return fail(HACK_ERR_INVALID_ARG, "sm_scale must be finite and non-negative");
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return fail(HACK_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
  if (cfg->dtype != HACK_F32 && cfg->dtype != HACK_BF16) return fail(HACK_ERR_UNSUPPORTED, "dtype must be HACK_F32 or HACK_BF16");
  if (cfg->n_obs < 1 || cfg->n_obs > hack::kMaxObs) return fail(HACK_ERR_UNSUPPORTED, "n_obs must be in 1..32");
  if (cfg->obs_sampler < HACK_OBS_UNIFORM || cfg->obs_sampler > HACK_OBS_FULL) return fail(HACK_ERR_INVALID_ARG, "unknown obs_sampler");
  if (cfg->merge_last != 0 && cfg->merge_last != 1) return fail(HACK_ERR_INVALID_ARG, "merge_last must be 0 or 1");
  if (cfg->merge_last && cfg->dtype != HACK_BF16) return fail(HACK_ERR_UNSUPPORTED, "merge_last needs a bf16 cache");
  for (int k = 0; k < cfg->n_scales; ++k)
    if (cfg->scale_sides[k] < 1 || cfg->scale_sides[k] > 1024) return fail(HACK_ERR_INVALID_ARG, "scale side out of range (1..1024)");
  for (int i = 0; i < cfg->n_layers * cfg->n_heads; ++i)
    if (cfg->head_is_contextual[i] > 1) return fail(HACK_ERR_INVALID_ARG, "head_is_contextual must hold 0 or 1");
  int n_dev = 0;
  HACK_CUDA(cudaGetDeviceCount(&n_dev));
  if (cfg->device < 0 || cfg->device >= n_dev) return fail(HACK_ERR_INVALID_ARG, "device ordinal out of range");
  HACK_CUDA(cudaSetDevice(cfg->device));

  hack_cache* c = new (std::nothrow) hack_cache();
  if (!c) return fail(HACK_ERR_OOM, "host allocation failed");
  c->cfg = *cfg;
  c->sides.assign(cfg->scale_sides, cfg->scale_sides + cfg->n_scales);
  c->mask.assign(cfg->head_is_contextual, cfg->head_is_contextual + (size_t)cfg->n_layers * cfg->n_heads);
  c->cfg.scale_sides = c->sides.data();
  c->cfg.head_is_contextual = c->mask.data();
  c->elt = cfg->dtype == HACK_F32 ? 4 : 2;
  c->budget[0] = cfg->budget_s;
  c->budget[1] = cfg->budget_c;
  c->sm_scale = cfg->sm_scale > 0.f ? cfg->sm_scale : 1.0f / std::sqrt((float)cfg->head_dim);
  long long cum = 0;
  for (int k = 0; k < cfg->n_scales; ++k) {
    c->n_tok.push_back(c->sides[k] * c->sides[k]);
    cum += c->n_tok[k];
    if (cum > (1ll << 28)) { delete c; return fail(HACK_ERR_UNSUPPORTED, "schedule too long"); }
    c->t_cum.push_back((int32_t)cum);
  }
  c->t_init = cfg->n_init_scales > 0 ? c->t_cum[cfg->n_init_scales - 1] : 0;
  // walk the schedule once to find capacities and buffer strides
  {
    LayerState ls;
    int cand_max = 1, kept_max = 1, new_max = 1;
    for (int k = 0; k < cfg->n_scales; ++k) {
      hack_step_info_t p;
      plan_step(c, ls, k, &p);
      cand_max = std::max({cand_max, p.cand_c, p.cand_s});
      kept_max = std::max({kept_max, p.kept_c, p.kept_s});
      new_max = std::max(new_max, p.n_new);
      c->cap[0] = std::max(c->cap[0], p.kept_s);
      c->cap[1] = std::max(c->cap[1], p.kept_c);
      ls.len[0] = p.kept_s;
      ls.len[1] = p.kept_c;
    }
    c->limits.cand_stride = (cand_max + 3) & ~3;
    c->limits.kept_stride = (kept_max + 3) & ~3;
    c->limits.max_new = new_max;
  }
  c->layers.assign(cfg->n_layers, LayerState());
  const int bh = cfg->batch * cfg->n_heads;
  std::vector<int32_t> row_off((size_t)cfg->n_layers * bh);
  size_t total_rows = 0;
  for (int l = 0; l < cfg->n_layers; ++l) {
    size_t rows = 0;
    int n_ctx = 0;
    for (int b = 0; b < cfg->batch; ++b)
      for (int h = 0; h < cfg->n_heads; ++h) {
        const int t = c->mask[(size_t)l * cfg->n_heads + h];
        row_off[(size_t)l * bh + b * cfg->n_heads + h] = (int32_t)rows;
        rows += c->cap[t] + kCanaryRows;            // checked builds: one guard row behind every head
        if (b == 0) n_ctx += t;
      }
    if (rows > (1ull << 30)) { delete c; return fail(HACK_ERR_UNSUPPORTED, "layer plane too large"); }
    c->n_ctx_heads.push_back(n_ctx);
    c->layer_rows.push_back(rows);
    c->layer_row_base.push_back(total_rows);
    total_rows += rows;
  }
  c->row_off_host = row_off;
  const size_t row_bytes = (size_t)cfg->head_dim * c->elt;
  const size_t pad_rows = 256;    // slack after the last layer so that tiled reads stay inside
  c->reserved_bytes = 2 * (total_rows - (size_t)kCanaryRows * cfg->n_layers * bh) * row_bytes;   // K and V rows proper

  auto bail = [&](hack_status_t s) { hack_free_cache(c); return s; };
#define HACK_TRY(call)                                                    \
  do {                                                                    \
    cudaError_t e_ = (call);                                              \
    if (e_ != cudaSuccess) {                                              \
      set_error(std::string(#call) + ": " + cudaGetErrorString(e_));      \
      return bail(e_ == cudaErrorMemoryAllocation ? HACK_ERR_OOM : HACK_ERR_CUDA); \
    }                                                                     \
  } while (0)
  HACK_TRY(cudaMalloc(&c->k_all, (total_rows + pad_rows) * row_bytes));
  HACK_TRY(cudaMalloc(&c->v_all, (total_rows + pad_rows) * row_bytes));
  HACK_TRY(cudaMalloc(&c->pos_all, (total_rows + pad_rows) * sizeof(int32_t)));
  HACK_TRY(cudaMemset(c->k_all, 0, (total_rows + pad_rows) * row_bytes));
  HACK_TRY(cudaMemset(c->v_all, 0, (total_rows + pad_rows) * row_bytes));
  HACK_TRY(cudaMemset(c->pos_all, 0, (total_rows + pad_rows) * sizeof(int32_t)));
  if (kCanaryRows) {
    // guard rows carry a byte pattern no kernel writes; hack_debug_check looks for it later
    for (int l = 0; l < cfg->n_layers; ++l)
      for (int i = 0; i < bh; ++i) {
        const int t = c->mask[(size_t)l * cfg->n_heads + i % cfg->n_heads];
        const size_t row = c->layer_row_base[l] + row_off[(size_t)l * bh + i] + c->cap[t];
        HACK_TRY(cudaMemset(c->k_all + row * row_bytes, hack::kCanaryByte, row_bytes));
        HACK_TRY(cudaMemset(c->v_all + row * row_bytes, hack::kCanaryByte, row_bytes));
        HACK_TRY(cudaMemset(c->pos_all + row, hack::kCanaryByte, sizeof(int32_t)));
      }
  }
  HACK_TRY(cudaMalloc(&c->row_off, row_off.size() * sizeof(int32_t)));
  HACK_TRY(cudaMemcpy(c->row_off, row_off.data(), row_off.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
  HACK_TRY(cudaMalloc(&c->mask_dev, c->mask.size()));
  HACK_TRY(cudaMemcpy(c->mask_dev, c->mask.data(), c->mask.size(), cudaMemcpyHostToDevice));
  HACK_TRY(cudaMalloc(&c->scores, (size_t)bh * c->limits.cand_stride * sizeof(float)));
  HACK_TRY(cudaMalloc(&c->idx, (size_t)bh * c->limits.kept_stride * sizeof(int32_t)));
  c->scratch.max_chunks = c->limits.cand_stride / hack::kScoreChunk + 2;   // stored part and new part are chunked separately
  HACK_TRY(cudaMalloc(&c->scratch.logits, (size_t)bh * hack::kMaxObs * c->limits.cand_stride * sizeof(float)));
  HACK_TRY(cudaMalloc(&c->scratch.partials, (size_t)bh * c->scratch.max_chunks * hack::kMaxObs * 2 * sizeof(float)));
  if (cfg->dtype == HACK_BF16) {
    // tensor maps of every layer's planes and the two head orders of the tensor-core attention
    c->k_maps.resize(cfg->n_layers);
    c->v_maps.resize(cfg->n_layers);
    std::vector<int32_t> order((size_t)cfg->n_layers * 2 * bh);
    for (int l = 0; l < cfg->n_layers; ++l) {
      const size_t rows = c->layer_rows[l] + (l + 1 == cfg->n_layers ? pad_rows : 0);
      if (!hack::make_rows_map(&c->k_maps[l], c->k_all + c->layer_row_base[l] * row_bytes, rows, cfg->head_dim) ||
          !hack::make_rows_map(&c->v_maps[l], c->v_all + c->layer_row_base[l] * row_bytes, rows, cfg->head_dim)) {
        set_error("cuTensorMapEncodeTiled failed for a cache plane");
        return bail(HACK_ERR_CUDA);
      }
      for (int first = 0; first < 2; ++first) {
        int32_t* o = order.data() + ((size_t)l * 2 + first) * bh;
        int n = 0;
        for (int pass = 0; pass < 2; ++pass)
          for (int i = 0; i < bh; ++i) {
            const int t = c->mask[(size_t)l * cfg->n_heads + i % cfg->n_heads];
            if ((pass == 0) == (t == first)) o[n++] = i;
          }
      }
    }
    HACK_TRY(cudaMalloc(&c->head_order, order.size() * sizeof(int32_t)));
    HACK_TRY(cudaMemcpy(c->head_order, order.data(), order.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
  }
  HACK_TRY(cudaMalloc(&c->n_old, (size_t)bh * sizeof(int32_t)));
  if (cfg->dtype == HACK_BF16) {
    c->var_blocks = c->limits.kept_stride / 128 + 1;
    HACK_TRY(cudaMalloc(&c->attn_row_stats, (size_t)bh * c->limits.max_new * 2 * sizeof(float)));
    HACK_TRY(cudaMalloc(&c->attn_block_var, (size_t)bh * c->var_blocks * sizeof(float)));
  }
  if (cfg->merge_last) {
    // what the contextual heads discard at the last scale
    LayerState ls;
    hack_step_info_t p{};
    for (int k = 0; k < cfg->n_scales; ++k) {
      plan_step(c, ls, k, &p);
      ls.len[0] = p.kept_s;
      ls.len[1] = p.kept_c;
    }
    hack::MergeScratch& m = c->merge;
    m.stride = ((std::max(p.cand_c - p.kept_c, 1) + 127) / 128) * 128;
    const size_t rows = (size_t)bh * m.stride;
    HACK_TRY(cudaMalloc(&m.ev_k, rows * row_bytes));
    HACK_TRY(cudaMalloc(&m.ev_v, rows * row_bytes));
    HACK_TRY(cudaMemset(m.ev_k, 0, rows * row_bytes));
    HACK_TRY(cudaMalloc(&m.ev_idx, rows * sizeof(int32_t)));
    HACK_TRY(cudaMalloc(&m.ev_inv_norm, rows * sizeof(float)));
    HACK_TRY(cudaMalloc(&m.kept_inv_norm, (size_t)bh * c->limits.kept_stride * sizeof(float)));
    HACK_TRY(cudaMalloc(&m.assign, rows * sizeof(int32_t)));
    HACK_TRY(cudaMalloc(&m.weight, rows * sizeof(float)));
    if (!hack::make_rows_map(&c->merge_ev_map, m.ev_k, rows, cfg->head_dim)) {
      set_error("cuTensorMapEncodeTiled failed for the merge scratch");
      return bail(HACK_ERR_CUDA);
    }
    m.ev_map = &c->merge_ev_map;
  }
  if (cfg->obs_sampler == HACK_OBS_CALLER) {
    HACK_TRY(cudaMalloc(&c->obs_rows, (size_t)cfg->n_scales * hack::kMaxObs * sizeof(int32_t)));
    HACK_TRY(cudaMemset(c->obs_rows, 0, (size_t)cfg->n_scales * hack::kMaxObs * sizeof(int32_t)));
    c->obs_rows_set.assign(cfg->n_scales, 0);
  }
  if (cfg->dtype == HACK_BF16) {
    HACK_TRY(cudaStreamCreateWithFlags(&c->side_stream, cudaStreamNonBlocking));
    HACK_TRY(cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming));
    HACK_TRY(cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming));
  }
  HACK_TRY(cudaMalloc(&c->status, sizeof(int)));
  HACK_TRY(cudaMemset(c->status, 0, sizeof(int)));
  HACK_TRY(cudaDeviceSynchronize());
#undef HACK_TRY
  *out = c;
  return HACK_OK;
}

hack_status_t hack_free_cache(hack_cache_t* c) {
  if (!c) return HACK_OK;
  cudaSetDevice(c->cfg.device);
  cudaDeviceSynchronize();
  cudaFree(c->k_all); cudaFree(c->v_all); cudaFree(c->pos_all); cudaFree(c->row_off);
  cudaFree(c->mask_dev); cudaFree(c->scores); cudaFree(c->idx);
  cudaFree(c->scratch.logits); cudaFree(c->scratch.partials); cudaFree(c->status);
  cudaFree(c->head_order);
  cudaFree(c->n_old);
  cudaFree(c->merge.ev_k);
  cudaFree(c->merge.ev_v);
  cudaFree(c->merge.ev_idx);
  cudaFree(c->merge.ev_inv_norm);
  cudaFree(c->merge.kept_inv_norm);
  cudaFree(c->merge.assign);
  cudaFree(c->merge.weight);
  cudaFree(c->attn_row_stats);
  cudaFree(c->attn_block_var);
  cudaFree(c->obs_rows);
  for (int sl = 0; sl < hack_cache::kHostSlots; ++sl) {
    for (int i = 0; i < 4; ++i) cudaFree(c->stage[sl][i]);
    if (c->ev_in[sl]) cudaEventDestroy(c->ev_in[sl]);
    if (c->ev_step[sl]) cudaEventDestroy(c->ev_step[sl]);
    if (c->ev_out[sl]) cudaEventDestroy(c->ev_out[sl]);
  }
  if (c->side_stream) cudaStreamDestroy(c->side_stream);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_join) cudaEventDestroy(c->ev_join);
  if (c->h2d_stream) cudaStreamDestroy(c->h2d_stream);
  if (c->d2h_stream) cudaStreamDestroy(c->d2h_stream);
  for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  delete c;
  return HACK_OK;
}

hack_status_t hack_set_obs_rows(hack_cache_t* c, int32_t scale, const int32_t* rows, int32_t n) {
  if (!c || !rows) return fail(HACK_ERR_INVALID_ARG, "cache or rows is NULL");
  if (c->cfg.obs_sampler != HACK_OBS_CALLER) return fail(HACK_ERR_STATE, "the cache was not created with HACK_OBS_CALLER");
  if (scale < 0 || scale >= c->cfg.n_scales) return fail(HACK_ERR_INVALID_ARG, "scale out of range");
  const int n_new = c->n_tok[scale];
  if (n != std::min(c->cfg.n_obs, n_new)) return fail(HACK_ERR_INVALID_ARG, "n must be min(N_obs, N_k)");
  for (int i = 0; i < n; ++i) {
    if (rows[i] < 0 || rows[i] >= n_new) return fail(HACK_ERR_INVALID_ARG, "observation row out of range");
    for (int j = 0; j < i; ++j)
      if (rows[j] == rows[i]) return fail(HACK_ERR_INVALID_ARG, "observation rows must be distinct");
  }
  HACK_CUDA(cudaSetDevice(c->cfg.device));
  HACK_CUDA(cudaMemcpy(c->obs_rows + (size_t)scale * hack::kMaxObs, rows, (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice));
  c->obs_rows_set[scale] = 1;
  return HACK_OK;
}

hack_status_t hack_reset(hack_cache_t* c) {
  if (!c) return fail(HACK_ERR_INVALID_ARG, "cache is NULL");
  for (auto& ls : c->layers) ls = LayerState();
  c->peak_bytes = 0;
  c->poisoned = false;
  return HACK_OK;
}

hack_status_t hack_get_limits(const hack_cache_t* c, hack_limits_t* out) {
  if (!c || !out) return fail(HACK_ERR_INVALID_ARG, "cache or out is NULL");
  *out = c->limits;
  return HACK_OK;
}

hack_status_t hack_step_info(const hack_cache_t* c, int32_t layer, int32_t scale, hack_step_info_t* out) {
  if (!out) return fail(HACK_ERR_INVALID_ARG, "out is NULL");
  if (!c) return fail(HACK_ERR_INVALID_ARG, "cache is NULL");
  if (layer < 0 || layer >= c->cfg.n_layers) return fail(HACK_ERR_INVALID_ARG, "layer out of range");
  if (scale < 0 || scale >= c->cfg.n_scales) return fail(HACK_ERR_INVALID_ARG, "scale out of range");
  const LayerState& ls = c->layers[layer];
  if (scale != ls.next_scale || ls.phase != 0) return fail(HACK_ERR_STATE, "scale is not this layer's next step");
  plan_step(c, ls, scale, out);
  return HACK_OK;
}

hack_status_t hack_score(hack_cache_t* c, int32_t layer, int32_t scale, const void* q,
                         const void* k_new, float* scores, void* stream) {
  hack_status_t s = check_step(c, layer, scale, 0);
  if (s != HACK_OK) return s;
  HACK_ON_DEVICE(c);
  if (!q || !k_new || !scores) return fail(HACK_ERR_INVALID_ARG, "q, k_new or scores is NULL");
  if (misaligned(q) || misaligned(k_new) || misaligned(scores)) return fail(HACK_ERR_INVALID_ARG, "buffers must be 16-byte aligned");
  hack_step_info_t p;
  plan_step(c, c->layers[layer], scale, &p);
  if (c->cfg.obs_sampler == HACK_OBS_CALLER && (p.triggered_c || p.triggered_s) && !c->obs_rows_set[scale])
    return fail(HACK_ERR_STATE, "HACK_OBS_CALLER: no observation rows were set for this scale (hack_set_obs_rows)");
  const hack::StepArgs a = make_args(c, layer, scale, p);
  StageScope ts(c, (cudaStream_t)stream, 0);
  int n = c->cfg.dtype == HACK_BF16
              ? hack::launch_compress_cluster(a, q, k_new, nullptr, scores, nullptr, (cudaStream_t)stream) : 0;
  if (n == 0) n = hack::launch_score(a, c->cfg.dtype, q, k_new, scores, c->scratch, (cudaStream_t)stream);
  if (n < 0) return HACK_ERR_CUDA;   // text recorded by the launcher
  ts.done(n);
  c->launches += n;
  return HACK_OK;
}

hack_status_t hack_select(hack_cache_t* c, int32_t layer, int32_t scale, const float* scores,
                          int32_t* idx, int32_t* kept_out, void* stream) {
  hack_status_t s = check_step(c, layer, scale, 0);
  if (s != HACK_OK) return s;
  HACK_ON_DEVICE(c);
  if (!scores || !idx) return fail(HACK_ERR_INVALID_ARG, "scores or idx is NULL");
  hack_step_info_t p;
  plan_step(c, c->layers[layer], scale, &p);
  const hack::StepArgs a = make_args(c, layer, scale, p);
  StageScope ts(c, (cudaStream_t)stream, 1);
  const int n = hack::launch_select(a, scores, idx, kept_out, (cudaStream_t)stream);
  if (n < 0) return HACK_ERR_CUDA;   // text recorded by the launcher
  ts.done(n);
  c->launches += n;
  return HACK_OK;
}

// Compaction of one step; with merge_last, at the last scale, wrapped in the merge of what the
// contextual heads discard.  Returns the number of launches, or -1.
static int compact_stage(hack_cache* c, const hack::StepArgs& a, const hack_step_info_t& p, int scale,
                         const int32_t* idx, int idx_all, const void* k_new, const void* v_new, cudaStream_t st) {
  const bool merge = c->cfg.merge_last && scale == c->cfg.n_scales - 1 && p.triggered_c && idx;
  int n = 0, r;
  if (merge) {
    if ((r = hack::launch_merge_prepare(a, c->merge, idx, k_new, v_new, st)) < 0) return -1;
    n += r;
  }
  if ((r = hack::launch_compact(a, c->cfg.dtype, idx, idx_all, k_new, v_new, st)) < 0) return -1;
  n += r;
  if (merge) {
    if ((r = hack::launch_merge_finish(a, c->merge, st)) < 0) return -1;
    n += r;
  }
  return n;
}

hack_status_t hack_compact(hack_cache_t* c, int32_t layer, int32_t scale, const int32_t* idx,
                           const void* k_new, const void* v_new, void* stream) {
  hack_status_t s = check_step(c, layer, scale, 0);
  if (s != HACK_OK) return s;
  HACK_ON_DEVICE(c);
  if (!idx || !k_new || !v_new) return fail(HACK_ERR_INVALID_ARG, "idx, k_new or v_new is NULL");
  if (misaligned(k_new) || misaligned(v_new)) return fail(HACK_ERR_INVALID_ARG, "buffers must be 16-byte aligned");
  hack_step_info_t p;
  plan_step(c, c->layers[layer], scale, &p);
  const hack::StepArgs a = make_args(c, layer, scale, p);
  StageScope ts(c, (cudaStream_t)stream, 2);
  const int n = compact_stage(c, a, p, scale, idx, 1, k_new, v_new, (cudaStream_t)stream);
  if (n < 0) return HACK_ERR_CUDA;   // text recorded by the launcher
  ts.done(n);
  c->launches += n;
  advance_after_compact(c, layer, p);
  return HACK_OK;
}

// k_new / v_new / seg_new: fused step only; head types flagged in seg_new have their new rows read
// from the caller's tensors and appended by the attention kernel itself.
static hack_status_t attend_impl(hack_cache* c, int layer, int scale, const void* q, void* out, float* sigma,
                                 cudaStream_t st, const void* k_new = nullptr, const void* v_new = nullptr,
                                 const int* seg_new = nullptr, int only_type = -1, bool finish = true,
                                 bool shares_gpu = false, bool follows_compression = false) {
  // lengths are already those after compaction
  LayerState& ls = c->layers[layer];
  hack_step_info_t p{};
  p.n_new = c->n_tok[scale];
  p.kept_s = ls.len[0];
  p.kept_c = ls.len[1];
  p.n_obs_rows = std::min(c->cfg.n_obs, p.n_new);
  hack::StepArgs a = make_args(c, layer, scale, p);
  if (seg_new) { a.seg_new[0] = seg_new[0]; a.seg_new[1] = seg_new[1]; }
  StageScope ts(c, st, 3);
  int n;
  if (sigma) {
    // Eq. 6 needs the statistics of every softmax row; the tensor-core attention kernel leaves them
    if (!hack::attend_tc_serves(a, c->cfg.dtype))
      return fail(HACK_ERR_UNSUPPORTED, "hack_attend_variance needs a bf16 cache and a scale of at least 32 tokens (128 query rows over all heads)");
    n = hack::launch_attend_tc(a, a.k_map, a.v_map, a.head_order, q, out, c->attn_row_stats, nullptr, nullptr, 0, false, st);
    if (n >= 0) {
      const int m = hack::launch_attention_variance(a, q, c->attn_row_stats, c->attn_block_var, c->var_blocks, sigma, st);
      n = m < 0 ? m : n + m;
    }
  } else if (seg_new) {
    int served = 0;
    if (only_type >= 0) {
      // the heads of one type: they lead the head order that puts that type first
      const int bh = c->cfg.batch * c->cfg.n_heads;
      const int n_ctx = c->cfg.batch * c->n_ctx_heads[layer];
      served = only_type == 1 ? n_ctx : bh - n_ctx;
      a.head_order = c->head_order + ((size_t)layer * 2 + only_type) * bh;
    }
    n = hack::launch_attend_tc(a, a.k_map, a.v_map, a.head_order, q, out, nullptr, k_new, v_new, served, shares_gpu, st,
                               follows_compression);
  } else {
    n = hack::launch_attend(a, c->cfg.dtype, q, out, st);
  }
  if (n < 0) return HACK_ERR_CUDA;   // text recorded by the launcher
  ts.done(n);
  c->launches += n;
  if (finish) {
    ls.phase = 0;
    ls.next_scale = scale + 1;
  }
  return HACK_OK;
}

hack_status_t hack_attend(hack_cache_t* c, int32_t layer, int32_t scale, const void* q, void* out, void* stream) {
  hack_status_t s = check_step(c, layer, scale, 1);
  if (s != HACK_OK) return s;
  HACK_ON_DEVICE(c);
  if (!q || !out) return fail(HACK_ERR_INVALID_ARG, "q or out is NULL");
  if (misaligned(q) || misaligned(out)) return fail(HACK_ERR_INVALID_ARG, "buffers must be 16-byte aligned");
  return attend_impl(c, layer, scale, q, out, nullptr, (cudaStream_t)stream);
}

hack_status_t hack_attend_variance(hack_cache_t* c, int32_t layer, int32_t scale, const void* q, void* out,
                                   float* sigma, void* stream) {
  hack_status_t s = check_step(c, layer, scale, 1);
  if (s != HACK_OK) return s;
  HACK_ON_DEVICE(c);
  if (!q || !out || !sigma) return fail(HACK_ERR_INVALID_ARG, "q, out or sigma is NULL");
  if (misaligned(q) || misaligned(out)) return fail(HACK_ERR_INVALID_ARG, "buffers must be 16-byte aligned");
  return attend_impl(c, layer, scale, q, out, sigma, (cudaStream_t)stream);
}

hack_status_t hack_classify_heads(const double* sigma, int32_t n_layers, int32_t n_heads, double alpha,
                                  uint8_t* head_is_contextual) {
  if (!sigma || !head_is_contextual) return fail(HACK_ERR_INVALID_ARG, "sigma or head_is_contextual is NULL");
  if (n_layers < 1 || n_heads < 1) return fail(HACK_ERR_INVALID_ARG, "n_layers and n_heads must be positive");
  if (!(alpha >= 0.0 && alpha <= 1.0)) return fail(HACK_ERR_INVALID_ARG, "alpha must be in [0, 1]");
  const int n = n_layers * n_heads;
  for (int i = 0; i < n; ++i)
    if (!std::isfinite(sigma[i])) return fail(HACK_ERR_INVALID_ARG, "sigma must be finite");
  std::vector<int> order(n);
  for (int i = 0; i < n; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return sigma[x] < sigma[y]; });
  const int n_ctx = (int)std::floor(alpha * n + 0.5);
  for (int i = 0; i < n; ++i) head_is_contextual[i] = 0;
  for (int i = 0; i < n_ctx; ++i) head_is_contextual[order[i]] = 1;
  return HACK_OK;
}

hack_status_t hack_scale_step(hack_cache_t* c, int32_t layer, int32_t scale, const void* q,
                              const void* k, const void* v, void* out, void* stream) {
  hack_status_t s = check_step(c, layer, scale, 0);
  if (s != HACK_OK) return s;
  HACK_ON_DEVICE(c);
  if (!q || !k || !v || !out) return fail(HACK_ERR_INVALID_ARG, "q, k, v or out is NULL");
  if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(out)) return fail(HACK_ERR_INVALID_ARG, "buffers must be 16-byte aligned");
  cudaStream_t st = (cudaStream_t)stream;
  hack_step_info_t p;
  plan_step(c, c->layers[layer], scale, &p);
  if (c->cfg.obs_sampler == HACK_OBS_CALLER && (p.triggered_c || p.triggered_s) && !c->obs_rows_set[scale])
    return fail(HACK_ERR_STATE, "HACK_OBS_CALLER: no observation rows were set for this scale (hack_set_obs_rows)");
  hack::StepArgs a = make_args(c, layer, scale, p);
  const bool any = p.triggered_c || p.triggered_s;
  int n = 0, r;
  // Tensor-core attention takes the rows of a head type that keeps the whole new scale straight
  // from the caller's K/V and appends them itself: types that evict nothing in this step, and
  // structural heads whose latest scale is protected (Eq. 11).  Contextual heads that evict rank the
  // new rows as well (Eq. 10) and are compacted first.  The final-scale merge keeps the separate
  // compaction it is wrapped around.
  const bool merge_step = c->cfg.merge_last && scale == c->cfg.n_scales - 1 && p.triggered_c;
  int seg_new[2] = {0, 0};
  const bool fused_append = hack::attend_tc_serves(a, c->cfg.dtype) && !merge_step;
  if (fused_append) {
    seg_new[0] = !p.triggered_s || a.protect_new;
    seg_new[1] = !p.triggered_c;
    a.seg_new[0] = seg_new[0];
    a.seg_new[1] = seg_new[1];
  }
  if (!any && p.n_new <= hack::kSmallQueries) {
    // nothing is evicted and the scale is small: one launch appends and attends
    StageScope ts(c, st, 3);
    if ((r = hack::launch_append_attend_small(a, c->cfg.dtype, q, k, v, out, st)) < 0) return HACK_ERR_CUDA;
    ts.done(r);
    c->launches += r;
    advance_after_compact(c, layer, p);
    LayerState& ls = c->layers[layer];
    ls.phase = 0;
    ls.next_scale = scale + 1;
    return HACK_OK;
  }
  bool compressed = false;
  // One head type compresses, the other only appends: the attention of the appending heads does
  // not depend on the compression, so it is enqueued on the cache's side stream, forked here (before
  // the compression launch) and joined at the end of the step.  Every (batch, head) is independent,
  // the two launches touch disjoint heads.
  const int n_ctx_bh = c->cfg.batch * c->n_ctx_heads[layer];
  const int n_heads_of[2] = {c->cfg.batch * c->cfg.n_heads - n_ctx_bh, n_ctx_bh};
  const int trig_type = p.triggered_c ? 1 : 0;
  const bool can_fork = any && fused_append && p.triggered_c != p.triggered_s && !c->timing && c->side_stream &&
                        n_heads_of[0] > 0 && n_heads_of[1] > 0;
  if (can_fork) {
    HACK_CUDA(cudaEventRecord(c->ev_fork, st));
    HACK_CUDA(cudaStreamWaitEvent(c->side_stream, c->ev_fork, 0));
  }
  if (any && fused_append) {
    // score, select and compact in one cluster launch per head (counted with the scoring stage)
    StageScope ts(c, st, 0);
    // the appending heads' attention (two query tiles per CTA) runs beside this launch
    const int beside = can_fork ? n_heads_of[1 - trig_type] * ((p.n_new + 255) / 256) : 0;
    if ((r = hack::launch_compress_cluster(a, q, k, v, nullptr, c->idx, st, beside)) < 0) return HACK_ERR_CUDA;
    ts.done(r);
    n += r;
    compressed = r > 0;
  }
  if (can_fork) {
    if (compressed) {
      c->launches += n;
      advance_after_compact(c, layer, p);
      s = attend_impl(c, layer, scale, q, out, nullptr, c->side_stream, k, v, seg_new, 1 - trig_type, false, true);
      if (s == HACK_OK) s = attend_impl(c, layer, scale, q, out, nullptr, st, k, v, seg_new, trig_type, true, false, true);
    }
    // the side stream always comes back to the caller's stream (it may be part of a capture)
    cudaEventRecord(c->ev_join, c->side_stream);
    cudaStreamWaitEvent(st, c->ev_join, 0);
    if (compressed) {
      if (s == HACK_ERR_CUDA) c->poisoned = true;
      return s;
    }
  }
  if (any && !compressed) {
    {
      StageScope ts(c, st, 0);
      if ((r = hack::launch_score(a, c->cfg.dtype, q, k, c->scores, c->scratch, st)) < 0) return HACK_ERR_CUDA;   // text recorded by the launcher
      ts.done(r);
      n += r;
    }
    {
      StageScope ts(c, st, 1);
      if ((r = hack::launch_select(a, c->scores, c->idx, nullptr, st)) < 0) return poison(c);
      ts.done(r);
      n += r;
    }
  }
  if ((any && !compressed) || !fused_append) {      // a step that only appends needs no launch ahead of the fused attention
    StageScope ts(c, st, 2);
    if ((r = compact_stage(c, a, p, scale, any ? c->idx : nullptr, any ? 1 : 0, k, v, st)) < 0) return any ? poison(c) : HACK_ERR_CUDA;
    ts.done(r);
    n += r;
  }
  c->launches += n;
  advance_after_compact(c, layer, p);
  s = attend_impl(c, layer, scale, q, out, nullptr, st, k, v, fused_append ? seg_new : nullptr, -1, true, false,
                  fused_append && compressed);
  if (s == HACK_ERR_CUDA) c->poisoned = true;     // compacted, attention not enqueued
  return s;
}

hack_status_t hack_scale_step_host(hack_cache_t* c, int32_t layer, int32_t scale, const void* q_host,
                                   const void* k_host, const void* v_host, void* out_host, void* stream) {
  hack_status_t s = check_step(c, layer, scale, 0);
  if (s != HACK_OK) return s;
  HACK_ON_DEVICE(c);
  if (!q_host || !k_host || !v_host || !out_host) return fail(HACK_ERR_INVALID_ARG, "a host buffer is NULL");
  cudaStream_t st = (cudaStream_t)stream;
  const size_t full = (size_t)c->cfg.batch * c->cfg.n_heads * c->limits.max_new * c->cfg.head_dim * c->elt;
  if (!c->h2d_stream) {
    // first use: staging sets, the two copy streams and the events that order them
    cudaError_t e = cudaStreamCreateWithFlags(&c->h2d_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->d2h_stream, cudaStreamNonBlocking);
    for (int sl = 0; sl < hack_cache::kHostSlots && e == cudaSuccess; ++sl) {
      for (int i = 0; i < 4 && e == cudaSuccess; ++i) e = cudaMalloc(&c->stage[sl][i], full);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_in[sl], cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_step[sl], cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_out[sl], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
      set_error(std::string("staging set-up: ") + cudaGetErrorString(e));
      cudaGetLastError();
      for (int sl = 0; sl < hack_cache::kHostSlots; ++sl) {
        for (int i = 0; i < 4; ++i) { cudaFree(c->stage[sl][i]); c->stage[sl][i] = nullptr; }
        if (c->ev_in[sl]) { cudaEventDestroy(c->ev_in[sl]); c->ev_in[sl] = nullptr; }
        if (c->ev_step[sl]) { cudaEventDestroy(c->ev_step[sl]); c->ev_step[sl] = nullptr; }
        if (c->ev_out[sl]) { cudaEventDestroy(c->ev_out[sl]); c->ev_out[sl] = nullptr; }
      }
      if (c->h2d_stream) { cudaStreamDestroy(c->h2d_stream); c->h2d_stream = nullptr; }
      if (c->d2h_stream) { cudaStreamDestroy(c->d2h_stream); c->d2h_stream = nullptr; }
      return e == cudaErrorMemoryAllocation ? HACK_ERR_OOM : HACK_ERR_CUDA;
    }
  }
  const int sl = (int)(c->host_calls % hack_cache::kHostSlots);
  const bool reused = c->host_calls >= (uint64_t)hack_cache::kHostSlots;
  unsigned char** sg = c->stage[sl];
  const size_t bytes = (size_t)c->cfg.batch * c->cfg.n_heads * c->n_tok[scale] * c->cfg.head_dim * c->elt;
  // upload: after the step that last read this staging set, not after anything else on `stream`
  if (reused) HACK_CUDA(cudaStreamWaitEvent(c->h2d_stream, c->ev_step[sl], 0));
  HACK_CUDA(cudaMemcpyAsync(sg[0], q_host, bytes, cudaMemcpyHostToDevice, c->h2d_stream));
  HACK_CUDA(cudaMemcpyAsync(sg[1], k_host, bytes, cudaMemcpyHostToDevice, c->h2d_stream));
  HACK_CUDA(cudaMemcpyAsync(sg[2], v_host, bytes, cudaMemcpyHostToDevice, c->h2d_stream));
  HACK_CUDA(cudaEventRecord(c->ev_in[sl], c->h2d_stream));
  // the step, on the caller's stream (the output staging buffer is free: the stream waited for
  // its download at the end of the call that used it)
  HACK_CUDA(cudaStreamWaitEvent(st, c->ev_in[sl], 0));
  s = hack_scale_step(c, layer, scale, sg[0], sg[1], sg[2], sg[3], stream);
  if (s != HACK_OK) return s;
  HACK_CUDA(cudaEventRecord(c->ev_step[sl], st));
  // download on its own stream; the caller's stream joins it, so that synchronising `stream`
  // still means out_host is complete
  HACK_CUDA(cudaStreamWaitEvent(c->d2h_stream, c->ev_step[sl], 0));
  HACK_CUDA(cudaMemcpyAsync(out_host, sg[3], bytes, cudaMemcpyDeviceToHost, c->d2h_stream));
  HACK_CUDA(cudaEventRecord(c->ev_out[sl], c->d2h_stream));
  HACK_CUDA(cudaStreamWaitEvent(st, c->ev_out[sl], 0));
  ++c->host_calls;
  return HACK_OK;
}

hack_status_t hack_get_lengths(const hack_cache_t* c, int32_t layer, int32_t* host_out) {
  if (!c || !host_out) return fail(HACK_ERR_INVALID_ARG, "cache or host_out is NULL");
  if (layer < 0 || layer >= c->cfg.n_layers) return fail(HACK_ERR_INVALID_ARG, "layer out of range");
  const LayerState& ls = c->layers[layer];
  for (int b = 0; b < c->cfg.batch; ++b)
    for (int h = 0; h < c->cfg.n_heads; ++h)
      host_out[b * c->cfg.n_heads + h] = ls.len[c->mask[(size_t)layer * c->cfg.n_heads + h]];
  return HACK_OK;
}

hack_status_t hack_read_head(hack_cache_t* c, int32_t layer, int32_t b, int32_t h, int32_t which,
                             void* host_out, size_t bytes) {
  if (!c || !host_out) return fail(HACK_ERR_INVALID_ARG, "cache or host_out is NULL");
  if (layer < 0 || layer >= c->cfg.n_layers || b < 0 || b >= c->cfg.batch || h < 0 || h >= c->cfg.n_heads)
    return fail(HACK_ERR_INVALID_ARG, "layer, b or h out of range");
  if (which < 0 || which > 2) return fail(HACK_ERR_INVALID_ARG, "which must be 0, 1 or 2");
  const int t = c->mask[(size_t)layer * c->cfg.n_heads + h];
  const size_t len = c->layers[layer].len[t];
  const size_t row_bytes = (size_t)c->cfg.head_dim * c->elt;
  const size_t need = which == 2 ? len * sizeof(int32_t) : len * row_bytes;
  if (bytes < need) return fail(HACK_ERR_INVALID_ARG, "host_out is too small for the stored length");
  const size_t off = c->row_off_host[((size_t)layer * c->cfg.batch + b) * c->cfg.n_heads + h];
  HACK_ON_DEVICE(c);
  HACK_CUDA(cudaDeviceSynchronize());
  const size_t row = c->layer_row_base[layer] + off;
  if (need == 0) return HACK_OK;
  if (which == 2) HACK_CUDA(cudaMemcpy(host_out, c->pos_all + row, need, cudaMemcpyDeviceToHost));
  else HACK_CUDA(cudaMemcpy(host_out, (which == 0 ? c->k_all : c->v_all) + row * row_bytes, need, cudaMemcpyDeviceToHost));
  return HACK_OK;
}

hack_status_t hack_kv_bytes(const hack_cache_t* c, size_t* live, size_t* peak, size_t* reserved) {
  if (!c) return fail(HACK_ERR_INVALID_ARG, "cache is NULL");
  if (live) *live = live_bytes(c);
  if (peak) *peak = c->peak_bytes;
  if (reserved) *reserved = c->reserved_bytes;
  return HACK_OK;
}

hack_status_t hack_launch_count(const hack_cache_t* c, uint64_t* launches) {
  if (!c || !launches) return fail(HACK_ERR_INVALID_ARG, "cache or launches is NULL");
  *launches = c->launches;
  return HACK_OK;
}

hack_status_t hack_stage_timing(hack_cache_t* c, int32_t enable) {
  if (!c) return fail(HACK_ERR_INVALID_ARG, "cache is NULL");
  HACK_ON_DEVICE(c);
  HACK_CUDA(cudaDeviceSynchronize());
  c->timing = enable != 0;
  c->spans.clear();
  c->ev_used = 0;
  for (int i = 0; i < 4; ++i) { c->stage_ms[i] = 0; c->stage_launches[i] = 0; }
  return HACK_OK;
}

hack_status_t hack_stage_times(hack_cache_t* c, double* ms, uint64_t* launches) {
  if (!c || !ms || !launches) return fail(HACK_ERR_INVALID_ARG, "cache, ms or launches is NULL");
  HACK_ON_DEVICE(c);
  HACK_CUDA(cudaDeviceSynchronize());
  for (const auto& sp : c->spans) {
    float t = 0.f;
    HACK_CUDA(cudaEventElapsedTime(&t, c->ev_pool[sp.e0], c->ev_pool[sp.e1]));
    c->stage_ms[sp.stage] += t;
    c->stage_launches[sp.stage] += sp.launches;
  }
  c->spans.clear();
  c->ev_used = 0;
  for (int i = 0; i < 4; ++i) { ms[i] = c->stage_ms[i]; launches[i] = c->stage_launches[i]; }
  return HACK_OK;
}

hack_status_t hack_set_wait_limit(hack_cache_t* c, int64_t cycles) {
  if (!c) return fail(HACK_ERR_INVALID_ARG, "cache is NULL");
  if (cycles < 0) return fail(HACK_ERR_INVALID_ARG, "the wait limit must not be negative");
  c->wait_cycles = cycles == 0 ? hack::kDefaultWaitCycles : (long long)cycles;
  return HACK_OK;
}

hack_status_t hack_poll_status(hack_cache_t* c, void* stream) {
  if (!c) return fail(HACK_ERR_INVALID_ARG, "cache is NULL");
  HACK_ON_DEVICE(c);
  HACK_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  int word = 0;
  HACK_CUDA(cudaMemcpy(&word, c->status, sizeof(int), cudaMemcpyDeviceToHost));
  if (word != 0) {
    HACK_CUDA(cudaMemset(c->status, 0, sizeof(int)));
    if (word >= hack::kDebugCodeBase) {
      set_error("checked build: bounds check " + std::to_string(word - hack::kDebugCodeBase) + " failed in a kernel (the access was skipped)");
      return HACK_ERR_STATE;
    }
    set_error("a bounded device-side wait expired (status word " + std::to_string(word) + ")");
    return HACK_ERR_TIMEOUT;
  }
  return HACK_OK;
}

hack_status_t hack_debug_check(hack_cache_t* c, int32_t* violations) {
  if (!c || !violations) return fail(HACK_ERR_INVALID_ARG, "cache or violations is NULL");
  *violations = 0;
  if (!kCanaryRows) return fail(HACK_ERR_UNSUPPORTED, "this library was built without HACK_DEBUG_CHECKS");
  HACK_ON_DEVICE(c);
  HACK_CUDA(cudaDeviceSynchronize());
  const int bh = c->cfg.batch * c->cfg.n_heads;
  const size_t row_bytes = (size_t)c->cfg.head_dim * c->elt;
  std::vector<unsigned char> row(row_bytes);
  int bad = 0;
  for (int l = 0; l < c->cfg.n_layers; ++l)
    for (int i = 0; i < bh; ++i) {
      const int t = c->mask[(size_t)l * c->cfg.n_heads + i % c->cfg.n_heads];
      const size_t r = c->layer_row_base[l] + c->row_off_host[(size_t)l * bh + i] + c->cap[t];
      for (int which = 0; which < 3; ++which) {
        const size_t n = which == 2 ? sizeof(int32_t) : row_bytes;
        const unsigned char* src = which == 0 ? c->k_all + r * row_bytes
                                  : which == 1 ? c->v_all + r * row_bytes
                                               : reinterpret_cast<const unsigned char*>(c->pos_all + r);
        HACK_CUDA(cudaMemcpy(row.data(), src, n, cudaMemcpyDeviceToHost));
        bool hit = false;
        for (size_t x = 0; x < n; ++x) hit = hit || row[x] != hack::kCanaryByte;
        if (hit) {
          if (bad == 0)
            set_error("canary row overwritten: layer " + std::to_string(l) + ", (batch, head) " + std::to_string(i) +
                      (which == 0 ? ", K plane" : which == 1 ? ", V plane" : ", position plane"));
          ++bad;
        }
      }
    }
  *violations = bad;
  return HACK_OK;
}

int32_t hack_debug_build(void) { return kCanaryRows; }

}  // extern "C"
