// Host side of the C ABI: argument validation, workspace layout, context bookkeeping.
// All device work is delegated to the launchers of the other translation units.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>

#include "d2o_common.cuh"

using namespace d2o;

static thread_local char g_cuda_err[256] = "";

static d2o_status cuda_fail(cudaError_t e, const char* where) {
  snprintf(g_cuda_err, sizeof(g_cuda_err), "%.160s: %.80s", where, cudaGetErrorString(e));
  return D2O_ERR_CUDA;
}
namespace d2o {
d2o_status record_cuda_error(cudaError_t e, const char* where) { return cuda_fail(e, where); }
}
#define CUDA_TRY(expr)                                   \
  do {                                                   \
    cudaError_t e_ = (expr);                             \
    if (e_ != cudaSuccess) return cuda_fail(e_, #expr);  \
  } while (0)

extern "C" const char* d2o_status_string(d2o_status s) {
  switch (s) {
    case D2O_OK: return "ok";
    case D2O_ERR_INVALID_ARG: return "invalid argument";
    case D2O_ERR_UNSUPPORTED: return "unsupported configuration";
    case D2O_ERR_WORKSPACE: return "workspace too small or misaligned";
    case D2O_ERR_STATE: return "call out of order";
    case D2O_ERR_CUDA: return "CUDA runtime error";
    case D2O_ERR_TIMEOUT: return "device-side wait ran out";
    case D2O_ERR_TOO_LARGE: return "problem exceeds the fixed capacity of the allocation-free entry point";
  }
  return "unknown status";
}

extern "C" const char* d2o_last_cuda_error(void) { return g_cuda_err; }

static int elem_size_of(int dtype) { return dtype == D2O_F32 ? 4 : 2; }
constexpr int kMaxSliceRows = 56 * 1024;      // rows of one slice (S_l + 1): 4 bytes each of the 227 KB of shared memory

static d2o_status validate(const d2o_config* c, int64_t* total_budget, int* max_budget) {
  if (!c) return D2O_ERR_INVALID_ARG;
  if (c->n_layers < 1 || c->n_layers > 1024 || c->batch < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1)
    return D2O_ERR_INVALID_ARG;
  if (c->n_q_heads % c->n_kv_heads != 0) return D2O_ERR_INVALID_ARG;
  int g = c->n_q_heads / c->n_kv_heads;
  if (g != 1 && g != 2 && g != 4 && g != 8) return D2O_ERR_UNSUPPORTED;
  if (c->d_head != 64 && c->d_head != 128) return D2O_ERR_UNSUPPORTED;
  if (c->dtype != D2O_F32 && c->dtype != D2O_F16 && c->dtype != D2O_BF16) return D2O_ERR_UNSUPPORTED;
  if (c->prompt_len < 1 || c->prompt_len > (1 << 20) || c->max_new_tokens < 0) return D2O_ERR_INVALID_ARG;
  if (!(c->rho > 0.0f) || !isfinite(c->rho)) return D2O_ERR_INVALID_ARG;
  if (c->n_sink < 0 || c->nm_ratio < 0.0f || !isfinite(c->nm_ratio)) return D2O_ERR_INVALID_ARG;
  if (!(c->beta >= 0.0f && c->beta <= 1.0f)) return D2O_ERR_INVALID_ARG;
  if (!(c->density_temp > 0.0f) || !isfinite(c->density_temp)) return D2O_ERR_INVALID_ARG;
  if (c->head_reduce < 0 || c->head_reduce > 3) return D2O_ERR_UNSUPPORTED;
  if (c->budget_rule < 0 || c->budget_rule > 2) return D2O_ERR_UNSUPPORTED;
  if (c->sim_feature < 0 || c->sim_feature > 1 || c->merge_policy < 0 || c->merge_policy > 1) return D2O_ERR_UNSUPPORTED;
  // the value-feature ablation is built for the prompt stage; the decode kernel computes its cosines on the keys
  if (c->sim_feature == 1 && c->max_new_tokens > 0) return D2O_ERR_UNSUPPORTED;
  int maxb = c->max_budget > 0 ? c->max_budget : c->prompt_len;
  if (maxb > c->prompt_len + c->max_new_tokens) return D2O_ERR_INVALID_ARG;
  if (c->min_budget < 1 || c->min_budget < c->n_sink + 1 || c->min_budget > maxb) return D2O_ERR_INVALID_ARG;
  // cache rows per KV head and sequence, summed over the layers: fixed by rho (rules 0 and 1), or bounded by the
  // upper clamp (rule 2, whose total depends on the densities)
  double tot = floor((double)c->rho * (double)c->n_layers * (double)c->prompt_len + 0.5);
  if (c->budget_rule == 1) {
    // per-head sizes add up to round(rho * L * Hkv * P) per sequence; per KV head that is at most this many rows more
    // than the mean, so the pool is sized by the total over heads (see layouts)
    tot = floor((double)c->rho * ((double)c->n_layers * c->n_kv_heads) * (double)c->prompt_len + 0.5);
    if (tot < (double)c->n_layers * c->n_kv_heads * c->min_budget || tot > (double)c->n_layers * c->n_kv_heads * maxb)
      return D2O_ERR_INVALID_ARG;
    if ((size_t)c->n_layers * c->n_kv_heads > 4096) return D2O_ERR_UNSUPPORTED;   // work arrays of the budget kernel
  } else if (c->budget_rule == 2) {
    tot = (double)c->n_layers * maxb;
  } else if (tot < (double)c->n_layers * c->min_budget || tot > (double)c->n_layers * maxb) {
    return D2O_ERR_INVALID_ARG;
  }
  // the prompt-stage segment kernel keeps one counter per retained row of a slice in shared memory
  if (maxb + 1 > kMaxSliceRows) return D2O_ERR_UNSUPPORTED;
  *total_budget = (int64_t)tot;
  *max_budget = maxb;
  return D2O_OK;
}

static void layouts(const d2o_config* c, int64_t total_budget, int max_budget, Layout* l, ScratchLayout* s) {
  const size_t B = c->batch, L = c->n_layers, Hq = c->n_q_heads, Hkv = c->n_kv_heads, P = c->prompt_len;
  const size_t d = c->d_head, e = elem_size_of(c->dtype);
  // every slice starts at a multiple of 8 rows; total_budget counts rows per KV head (per-layer rules) or over all KV
  // heads (per-head rule) of one sequence
  const size_t rows = c->budget_rule == 1 ? B * ((size_t)total_budget + 7 * L * Hkv)
                                          : B * Hkv * ((size_t)total_budget + 7 * L);
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  l->status = take(16);
  l->counters = take(kNumCounters * 8);
  l->density = take(B * L * Hq * 8);
  l->budgets = take(B * L * Hkv * 4);
  l->windows = take(B * L * Hkv * 4);
  l->row_off = take(B * L * Hkv * 8);
  l->order = take(B * L * 4);
  l->plen = take(B * 4);
  l->len = take(L * B * Hkv * 4);
  l->tau = take(L * B * Hkv * 4);
  l->steps_done = take(L * B * Hkv * 4);
  l->sim_items = take(c->dtype == D2O_F32 ? 0 : L * sim_tc_max_items(c, max_budget) * 16);
  l->colsum = take(L * B * Hq * P * 4);
  l->pos = take(rows * 4);
  l->score = take(rows * 4);
  l->rnorm = take(rows * 4);
  l->kpool = take(rows * d * e);
  l->vpool = take(rows * d * e);
  l->end = o;
  o = 0;
  s->lse = take(B * Hq * P * 4);
  s->lse_stride = o - s->lse;
  o += (size_t)(kStatsLanes - 1) * s->lse_stride;
  s->evict_idx = take(B * Hkv * P * 4);
  s->evict_mx = take(B * Hkv * P * 4);
  s->evict_nn = take(B * Hkv * P * 4);
  s->seg_start = take(B * Hkv * ((size_t)max_budget + 2) * 4);
  s->seg_items = take(B * Hkv * P * 4);
  s->seg_tmp = take(B * Hkv * P * 4);
  s->part_key = take(c->dtype == D2O_F32 ? 0 : sim_tc_part_key_bytes(c, max_budget));
  s->lane_stride = o - s->evict_idx;                       // the arrays above, once more per further lane
  o += (size_t)(kCompressLanes - 1) * s->lane_stride;
  s->pl_spill = take((rows + 8 * L * B * Hkv) * (Hq / Hkv) * 4);
  s->stage_q = take(L * B * Hq * d * e);
  s->stage_k = take(L * B * Hkv * d * e);
  s->stage_v = take(L * B * Hkv * d * e);
  s->stage_out = take(L * B * Hq * d * e);
  s->stage_stride = o - s->stage_q;                        // further sets of the four for the pipelined host path
  o += (size_t)(2 * kHostBlock - 1) * s->stage_stride;
  s->end = o;
}

extern "C" d2o_status d2o_workspace_size(const d2o_config* cfg, size_t* state_bytes, size_t* scratch_bytes) {
  int64_t tot; int maxb;
  d2o_status st = validate(cfg, &tot, &maxb);
  if (st != D2O_OK) return st;
  if (!state_bytes || !scratch_bytes) return D2O_ERR_INVALID_ARG;
  Layout l; ScratchLayout s;
  layouts(cfg, tot, maxb, &l, &s);
  *state_bytes = l.end;
  *scratch_bytes = s.end;
  return D2O_OK;
}

extern "C" d2o_status d2o_create(const d2o_config* cfg, void* state, size_t state_bytes, void* scratch,
                                 size_t scratch_bytes, void* stream, d2o_ctx** out) {
  int64_t tot; int maxb;
  d2o_status st = validate(cfg, &tot, &maxb);
  if (st != D2O_OK) return st;
  if (!state || !scratch || !out) return D2O_ERR_INVALID_ARG;
  if (((uintptr_t)state & 255) || ((uintptr_t)scratch & 255)) return D2O_ERR_WORKSPACE;
  Layout l; ScratchLayout s;
  layouts(cfg, tot, maxb, &l, &s);
  if (state_bytes < l.end || scratch_bytes < s.end) return D2O_ERR_WORKSPACE;
  d2o_ctx* c = (d2o_ctx*)calloc(1, sizeof(d2o_ctx));
  if (!c) return D2O_ERR_INVALID_ARG;
  c->cfg = *cfg;
  c->group = cfg->n_q_heads / cfg->n_kv_heads;
  c->elem_size = elem_size_of(cfg->dtype);
  c->max_budget = maxb;
  c->total_budget = tot;
  c->pool_rows = cfg->budget_rule == 1
      ? (int64_t)cfg->batch * (tot + 7 * (int64_t)cfg->n_layers * cfg->n_kv_heads)
      : (int64_t)cfg->batch * cfg->n_kv_heads * (tot + 7 * (int64_t)cfg->n_layers);
  c->lay = l; c->slay = s;
  c->decode_l2_hints = 1;
  c->producer_stop_stage = -1;
  {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
      (void)cudaGetLastError();
      free(c);
      return D2O_ERR_CUDA;
    }
    c->n_sms = sms;
  }
  c->state = (char*)state; c->scratch = (char*)scratch;
  c->state_bytes = state_bytes; c->scratch_bytes = scratch_bytes;
  const size_t BL = (size_t)cfg->batch * cfg->n_layers;
  const size_t BLH = BL * cfg->n_kv_heads;
  c->h_budgets = (int32_t*)calloc(BLH, 4);
  c->h_windows = (int32_t*)calloc(BLH, 4);
  c->h_row_off = (int64_t*)calloc(BLH, 8);
  c->h_pair_max = (int32_t*)calloc(BL, 4);
  c->h_pair_sum = (int64_t*)calloc(BL, 8);
  c->layer_fed = (uint8_t*)calloc(cfg->n_layers, 1);
  c->layer_compressed = (uint8_t*)calloc(cfg->n_layers, 1);
  c->layer_steps = (int32_t*)calloc(cfg->n_layers, 4);
  c->h_order = (int32_t*)calloc(BL, 4);
  c->h_plen = (int32_t*)calloc(cfg->batch, 4);
  c->h_sim_count = (int32_t*)calloc(cfg->n_layers, 4);
  c->h_sim_items = cfg->dtype == D2O_F32 ? nullptr
      : (int4*)malloc((size_t)cfg->n_layers * sim_tc_max_items(cfg, maxb) * sizeof(int4));
  for (int b = 0; b < cfg->batch; ++b) c->h_plen[b] = cfg->prompt_len;
  // bookkeeping (status, counters, density, budgets ... tau) starts at zero
  cudaError_t e = cudaMemsetAsync(c->state, 0, l.colsum, (cudaStream_t)stream);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(c->state + l.plen, c->h_plen, (size_t)cfg->batch * 4, cudaMemcpyHostToDevice, (cudaStream_t)stream);
  if (e != cudaSuccess) { d2o_destroy(c); return cuda_fail(e, "cudaMemsetAsync(state)"); }
  *out = c;
  return D2O_OK;
}

extern "C" void d2o_destroy(d2o_ctx* c) {
  if (!c) return;
  if (c->io_ready) {
    cudaStreamDestroy(c->io_in); cudaStreamDestroy(c->io_out); cudaEventDestroy(c->io_start);
    for (int i = 0; i < 2; ++i) {
      cudaEventDestroy(c->io_in_done[i]); cudaEventDestroy(c->io_step_done[i]); cudaEventDestroy(c->io_out_done[i]);
    }
  }
  if (c->lanes_ready) {
    for (int i = 0; i < kCompressLanes; ++i) { cudaStreamDestroy(c->lane_stream[i]); cudaEventDestroy(c->lane_done[i]); }
    cudaEventDestroy(c->lane_fork);
  }
  free(c->h_budgets); free(c->h_windows); free(c->h_row_off); free(c->h_pair_max); free(c->h_pair_sum);
  free(c->layer_fed); free(c->layer_compressed); free(c->layer_steps); free(c->h_order); free(c->h_plen); free(c->h_sim_count); free(c->h_sim_items);
  free(c);
}

static bool aligned16(const void* p) { return p && (((uintptr_t)p & 15) == 0); }

extern "C" d2o_status d2o_layer_stats(d2o_ctx* c, int32_t layer, const void* Q, const void* K, const float* lse,
                                      void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return D2O_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || (lse && !aligned16(lse))) return D2O_ERR_INVALID_ARG;
  CUDA_TRY(launch_layer_stats(c, layer, Q, K, lse, (cudaStream_t)stream));
  c->layer_fed[layer] = 1;
  return D2O_OK;
}

// the library's own streams for the multi-layer calls: streams and events only, no device memory
static d2o_status ensure_lanes(d2o_ctx* c) {
  if (c->lanes_ready) return D2O_OK;
  for (int i = 0; i < kCompressLanes; ++i) {
    CUDA_TRY(cudaStreamCreateWithFlags(&c->lane_stream[i], cudaStreamNonBlocking));
    CUDA_TRY(cudaEventCreateWithFlags(&c->lane_done[i], cudaEventDisableTiming));
  }
  CUDA_TRY(cudaEventCreateWithFlags(&c->lane_fork, cudaEventDisableTiming));
  c->lanes_ready = true;
  return D2O_OK;
}

extern "C" d2o_status d2o_layer_stats_layers(d2o_ctx* c, int32_t l0, int32_t l1, const void* const* Q,
                                             const void* const* K, const float* const* lse, void* stream) {
  if (!c || !Q || !K || l0 < 0 || l1 > c->cfg.n_layers || l0 >= l1) return D2O_ERR_INVALID_ARG;
  for (int l = l0; l < l1; ++l)
    if (!aligned16(Q[l - l0]) || !aligned16(K[l - l0]) || (lse && lse[l - l0] && !aligned16(lse[l - l0])))
      return D2O_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (l1 - l0 == 1) {
    CUDA_TRY(launch_layer_stats(c, l0, Q[0], K[0], lse ? lse[0] : nullptr, st));
  } else {
    const d2o_status ls = ensure_lanes(c);
    if (ls != D2O_OK) return ls;
    const int lanes = min(kStatsLanes, l1 - l0);
    CUDA_TRY(cudaEventRecord(c->lane_fork, st));
    for (int i = 0; i < lanes; ++i) CUDA_TRY(cudaStreamWaitEvent(c->lane_stream[i], c->lane_fork, 0));
    for (int l = l0; l < l1; ++l) {
      const int lane = (l - l0) % lanes;                     // a lane's layers follow one another on its stream
      CUDA_TRY(launch_layer_stats(c, l, Q[l - l0], K[l - l0], lse ? lse[l - l0] : nullptr, c->lane_stream[lane], lane));
    }
    for (int i = 0; i < lanes; ++i) {
      CUDA_TRY(cudaEventRecord(c->lane_done[i], c->lane_stream[i]));
      CUDA_TRY(cudaStreamWaitEvent(st, c->lane_done[i], 0));
    }
  }
  for (int l = l0; l < l1; ++l) c->layer_fed[l] = 1;
  return D2O_OK;
}

extern "C" d2o_status d2o_budgets_from_density(const double* density, int32_t batch, int32_t n_layers,
                                               int32_t n_heads, int32_t n_kv_heads, int32_t prompt_len, float rho,
                                               int32_t min_budget, int32_t max_budget, float density_temp,
                                               int32_t head_reduce, int32_t budget_rule, int32_t n_sink,
                                               int32_t window, float nm_ratio, int32_t* budgets, int32_t* windows,
                                               int64_t* row_off, int32_t* status_word, void* stream) {
  if (!density || !budgets || batch < 1 || n_layers < 1 || n_layers > 1024 || n_heads < 1 || n_kv_heads < 1 ||
      prompt_len < 1 || n_heads % n_kv_heads != 0)
    return D2O_ERR_INVALID_ARG;
  if (!(rho > 0.0f) || !(density_temp > 0.0f) || head_reduce < 0 || head_reduce > 3) return D2O_ERR_INVALID_ARG;
  if (budget_rule < 0 || budget_rule > 2) return D2O_ERR_INVALID_ARG;
  if (max_budget <= 0) max_budget = prompt_len;
  if (min_budget < 1 || min_budget > max_budget) return D2O_ERR_INVALID_ARG;
  const double units = budget_rule == 1 ? (double)n_layers * n_kv_heads : (double)n_layers;
  if (units > 4096) return D2O_ERR_UNSUPPORTED;
  double tot = floor((double)rho * units * prompt_len + 0.5);
  if (budget_rule != 2 && (tot < units * min_budget || tot > units * max_budget)) return D2O_ERR_INVALID_ARG;
  CUDA_TRY(launch_budgets(density, batch, n_layers, n_heads, n_kv_heads, prompt_len, rho, min_budget, max_budget,
                          density_temp, head_reduce, budget_rule, n_sink, window, nm_ratio, budgets, windows, row_off,
                          (uint32_t*)status_word, nullptr, (cudaStream_t)stream));
  return D2O_OK;
}

extern "C" d2o_status d2o_layer_budgets(d2o_ctx* c, int32_t* budgets_host, void* stream) {
  if (!c) return D2O_ERR_INVALID_ARG;
  for (int l = 0; l < c->cfg.n_layers; ++l)
    if (!c->layer_fed[l]) return D2O_ERR_STATE;
  const d2o_config& g = c->cfg;
  cudaStream_t st = (cudaStream_t)stream;
  int32_t* d_b = (int32_t*)(c->state + c->lay.budgets);
  int32_t* d_w = (int32_t*)(c->state + c->lay.windows);
  int64_t* d_o = (int64_t*)(c->state + c->lay.row_off);
  CUDA_TRY(launch_budgets((const double*)(c->state + c->lay.density), g.batch, g.n_layers, g.n_q_heads,
                          g.n_kv_heads, g.prompt_len, g.rho, g.min_budget, g.max_budget, g.density_temp,
                          g.head_reduce, g.budget_rule, g.n_sink, g.window, g.nm_ratio, d_b, d_w, d_o,
                          (uint32_t*)(c->state + c->lay.status), (const int32_t*)(c->state + c->lay.plen), st));
  const size_t BL = (size_t)g.batch * g.n_layers;
  const size_t Hkv = g.n_kv_heads, BLH = BL * Hkv;
  CUDA_TRY(cudaMemcpyAsync(c->h_budgets, d_b, BLH * 4, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaMemcpyAsync(c->h_windows, d_w, BLH * 4, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaMemcpyAsync(c->h_row_off, d_o, BLH * 8, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  // the device computed offsets for the pool; make sure they fit what the caller gave us
  for (size_t i = 0; i < BLH; ++i) {
    int64_t end = c->h_row_off[i] + (int64_t)slice_stride(c->h_budgets[i]);
    if (c->h_budgets[i] < 1 || c->h_budgets[i] > c->max_budget || c->h_row_off[i] < 0 || end > c->pool_rows)
      return D2O_ERR_STATE;
  }
  // largest and summed cache size over the KV heads of every (sequence, layer) pair
  for (size_t i = 0; i < BL; ++i) {
    int32_t mx = 0; int64_t sm = 0;
    for (size_t h = 0; h < Hkv; ++h) { mx = std::max(mx, c->h_budgets[i * Hkv + h]); sm += c->h_budgets[i * Hkv + h]; }
    c->h_pair_max[i] = mx; c->h_pair_sum[i] = sm;
  }
  // (layer, sequence) pairs by cache size, largest first: the decode kernel takes its slices in this order
  for (size_t i = 0; i < BL; ++i) c->h_order[i] = (int32_t)i;                  // i = layer * B + b
  {
    const int Bn = g.batch, Ln = g.n_layers;
    const int32_t* hb = c->h_pair_max;                                           // [B, L]
    std::stable_sort(c->h_order, c->h_order + BL, [=](int32_t x, int32_t y) {
      return hb[(x % Bn) * Ln + x / Bn] > hb[(y % Bn) * Ln + y / Bn];
    });
  }
  CUDA_TRY(cudaMemcpyAsync(c->state + c->lay.order, c->h_order, BL * 4, cudaMemcpyHostToDevice, st));
  if (c->h_sim_items) {
    // work lists of the tensor-core similarity kernel for every layer (the budgets are all it needs)
    sim_tc_build_items(c, c->n_sms, c->h_sim_items, c->h_sim_count);
    CUDA_TRY(cudaMemcpyAsync(c->state + c->lay.sim_items, c->h_sim_items,
                             (size_t)g.n_layers * sim_tc_max_items(&g, c->max_budget) * sizeof(int4),
                             cudaMemcpyHostToDevice, st));
  }
  CUDA_TRY(cudaStreamSynchronize(st));
  c->have_budgets = true;
  if (budgets_host) memcpy(budgets_host, c->h_budgets, BLH * 4);
  return D2O_OK;
}

extern "C" d2o_status d2o_prefill_compress(d2o_ctx* c, int32_t layer, const void* K, const void* V, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return D2O_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V)) return D2O_ERR_INVALID_ARG;
  if (!c->have_budgets) return D2O_ERR_STATE;
  CUDA_TRY(launch_prefill_compress(c, layer, K, V, (cudaStream_t)stream));
  c->layer_compressed[layer] = 1;
  c->layer_steps[layer] = 0;
  return D2O_OK;
}

extern "C" d2o_status d2o_prefill_compress_layers(d2o_ctx* c, int32_t l0, int32_t l1, const void* const* K,
                                                  const void* const* V, void* stream) {
  if (!c || !K || !V || l0 < 0 || l1 > c->cfg.n_layers || l0 >= l1) return D2O_ERR_INVALID_ARG;
  for (int l = l0; l < l1; ++l)
    if (!aligned16(K[l - l0]) || !aligned16(V[l - l0])) return D2O_ERR_INVALID_ARG;
  if (!c->have_budgets) return D2O_ERR_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  if (l1 - l0 == 1) {
    CUDA_TRY(launch_prefill_compress(c, l0, K[0], V[0], st));
  } else {
    const d2o_status ls = ensure_lanes(c);
    if (ls != D2O_OK) return ls;
    // the lanes start behind everything the caller's stream holds, the caller's stream goes on behind every lane
    const int lanes = min(kCompressLanes, l1 - l0);
    CUDA_TRY(cudaEventRecord(c->lane_fork, st));
    for (int i = 0; i < lanes; ++i) CUDA_TRY(cudaStreamWaitEvent(c->lane_stream[i], c->lane_fork, 0));
    for (int l = l0; l < l1; ++l) {
      const int lane = (l - l0) % lanes;                     // a lane's layers follow one another on its stream
      CUDA_TRY(launch_prefill_compress(c, l, K[l - l0], V[l - l0], c->lane_stream[lane], lane));
    }
    for (int i = 0; i < lanes; ++i) {
      CUDA_TRY(cudaEventRecord(c->lane_done[i], c->lane_stream[i]));
      CUDA_TRY(cudaStreamWaitEvent(st, c->lane_done[i], 0));
    }
  }
  for (int l = l0; l < l1; ++l) { c->layer_compressed[l] = 1; c->layer_steps[l] = 0; }
  return D2O_OK;
}

static d2o_status check_decode_range(d2o_ctx* c, int l0, int l1) {
  if (!c || l0 < 0 || l1 > c->cfg.n_layers || l0 >= l1) return D2O_ERR_INVALID_ARG;
  for (int l = l0; l < l1; ++l) {
    if (!c->layer_compressed[l]) return D2O_ERR_STATE;
    if (c->layer_steps[l] != c->layer_steps[l0]) return D2O_ERR_STATE;
  }
  if (c->layer_steps[l0] >= c->cfg.max_new_tokens) return D2O_ERR_STATE;
  return D2O_OK;
}

extern "C" d2o_status d2o_decode_step(d2o_ctx* c, int32_t l0, int32_t l1, const void* q, const void* k,
                                      const void* v, void* out, void* stream) {
  d2o_status st = check_decode_range(c, l0, l1);
  if (st != D2O_OK) return st;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return D2O_ERR_INVALID_ARG;
  d2o_status why = D2O_OK;
  cudaError_t e = launch_decode(c, l0, l1, q, k, v, out, (cudaStream_t)stream, &why);
  if (why != D2O_OK) return why;
  if (e != cudaSuccess) return cuda_fail(e, "launch_decode");
  for (int l = l0; l < l1; ++l) c->layer_steps[l] += 1;
  return D2O_OK;
}

extern "C" d2o_status d2o_decode_steps(d2o_ctx* c, int32_t l0, int32_t l1, int32_t n_steps, const void* q,
                                       const void* k, const void* v, void* out, void* stream) {
  d2o_status st = check_decode_range(c, l0, l1);
  if (st != D2O_OK) return st;
  if (n_steps < 1) return D2O_ERR_INVALID_ARG;
  if (c->layer_steps[l0] + n_steps > c->cfg.max_new_tokens) return D2O_ERR_STATE;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return D2O_ERR_INVALID_ARG;
  const d2o_config& g = c->cfg;
  const size_t nl = (size_t)(l1 - l0);
  const size_t qb = nl * g.batch * g.n_q_heads * g.d_head * c->elem_size;     // bytes of one step's q and out
  const size_t kb = nl * g.batch * g.n_kv_heads * g.d_head * c->elem_size;    // of its k and v
  for (int s = 0; s < n_steps; ++s) {
    d2o_status why = D2O_OK;
    // the first step is ordered behind whatever the stream ran before; the later ones are chained to their predecessor
    cudaError_t e = launch_decode(c, l0, l1, (const char*)q + s * qb, (const char*)k + s * kb, (const char*)v + s * kb,
                                  (char*)out + s * qb, (cudaStream_t)stream, &why, s > 0, s + 1 < n_steps);
    if (why != D2O_OK) return why;
    if (e != cudaSuccess) return cuda_fail(e, "launch_decode");
    for (int l = l0; l < l1; ++l) c->layer_steps[l] += 1;
  }
  return D2O_OK;
}

extern "C" d2o_status d2o_decode_step_host(d2o_ctx* c, int32_t l0, int32_t l1, const void* q_host,
                                           const void* k_host, const void* v_host, void* out_host, void* stream) {
  d2o_status st = check_decode_range(c, l0, l1);
  if (st != D2O_OK) return st;
  if (!q_host || !k_host || !v_host || !out_host) return D2O_ERR_INVALID_ARG;
  const d2o_config& g = c->cfg;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t nl = (size_t)(l1 - l0);
  const size_t qb = nl * g.batch * g.n_q_heads * g.d_head * c->elem_size;
  const size_t kb = nl * g.batch * g.n_kv_heads * g.d_head * c->elem_size;
  char* dq = c->scratch + c->slay.stage_q;
  char* dk = c->scratch + c->slay.stage_k;
  char* dv = c->scratch + c->slay.stage_v;
  char* dout = c->scratch + c->slay.stage_out;
  // q, k, v adjacent in host memory (in this order) and in the staging area: one transfer instead of three.  The
  // runtime rejects a range that spans two separately pinned allocations before enqueuing anything; then, as for
  // buffers that are not adjacent, three transfers.
  const char* qh = (const char*)q_host;
  bool merged = false;
  if ((const char*)k_host == qh + qb && (const char*)v_host == qh + qb + kb && dk == dq + qb && dv == dk + kb) {
    merged = cudaMemcpyAsync(dq, q_host, qb + 2 * kb, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (!merged) (void)cudaGetLastError();
  }
  if (!merged) {
    CUDA_TRY(cudaMemcpyAsync(dq, q_host, qb, cudaMemcpyHostToDevice, s));
    CUDA_TRY(cudaMemcpyAsync(dk, k_host, kb, cudaMemcpyHostToDevice, s));
    CUDA_TRY(cudaMemcpyAsync(dv, v_host, kb, cudaMemcpyHostToDevice, s));
  }
  d2o_status why = D2O_OK;
  cudaError_t e = launch_decode(c, l0, l1, dq, dk, dv, dout, s, &why);
  if (why != D2O_OK) return why;
  if (e != cudaSuccess) return cuda_fail(e, "launch_decode");
  CUDA_TRY(cudaMemcpyAsync(out_host, dout, qb, cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaStreamSynchronize(s));
  for (int l = l0; l < l1; ++l) c->layer_steps[l] += 1;
  return D2O_OK;
}

extern "C" d2o_status d2o_decode_steps_host(d2o_ctx* c, int32_t l0, int32_t l1, int32_t n_steps, const void* q_host,
                                            const void* k_host, const void* v_host, void* out_host, void* stream) {
  d2o_status st = check_decode_range(c, l0, l1);
  if (st != D2O_OK) return st;
  if (n_steps < 1 || !q_host || !k_host || !v_host || !out_host) return D2O_ERR_INVALID_ARG;
  if (c->layer_steps[l0] + n_steps > c->cfg.max_new_tokens) return D2O_ERR_STATE;
  const d2o_config& g = c->cfg;
  cudaStream_t s = (cudaStream_t)stream;
  if (!c->io_ready) {
    // streams and events only: no device memory
    CUDA_TRY(cudaStreamCreateWithFlags(&c->io_in, cudaStreamNonBlocking));
    CUDA_TRY(cudaStreamCreateWithFlags(&c->io_out, cudaStreamNonBlocking));
    CUDA_TRY(cudaEventCreateWithFlags(&c->io_start, cudaEventDisableTiming));
    for (int i = 0; i < 2; ++i) {
      CUDA_TRY(cudaEventCreateWithFlags(&c->io_in_done[i], cudaEventDisableTiming));
      CUDA_TRY(cudaEventCreateWithFlags(&c->io_step_done[i], cudaEventDisableTiming));
      CUDA_TRY(cudaEventCreateWithFlags(&c->io_out_done[i], cudaEventDisableTiming));
    }
    c->io_ready = true;
  }
  const size_t nl = (size_t)(l1 - l0);
  const size_t qb = nl * g.batch * g.n_q_heads * g.d_head * c->elem_size;
  const size_t kb = nl * g.batch * g.n_kv_heads * g.d_head * c->elem_size;
  // Steps go in blocks of kHostBlock; block b uses the staging sets of parity b % 2.  Three streams: the copies of
  // block b + 1 to the device and of block b - 1 back run beside the kernels of block b.  Inside a block the inputs of
  // every step are on the device before its first step is launched, so its steps are chained like those of
  // d2o_decode_steps.  A parity's sets are refilled once the block that read them is done (io_step_done), and their
  // outputs are overwritten once the copies back of the block before last are done (io_out_done).
  CUDA_TRY(cudaEventRecord(c->io_start, s));
  CUDA_TRY(cudaStreamWaitEvent(c->io_in, c->io_start, 0));
  CUDA_TRY(cudaStreamWaitEvent(c->io_out, c->io_start, 0));
  const int n_blocks = (n_steps + kHostBlock - 1) / kHostBlock;
  for (int b = 0; b < n_blocks; ++b) {
    const int par = b & 1, t0 = b * kHostBlock, cnt = min(kHostBlock, n_steps - t0);
    auto set_base = [&](int i) { return c->scratch + (size_t)(par * kHostBlock + i) * c->slay.stage_stride; };
    if (b >= 2) CUDA_TRY(cudaStreamWaitEvent(c->io_in, c->io_step_done[par], 0));
    for (int i = 0; i < cnt; ++i) {
      char* base = set_base(i);
      const size_t t = (size_t)(t0 + i);
      CUDA_TRY(cudaMemcpyAsync(base + c->slay.stage_q, (const char*)q_host + t * qb, qb, cudaMemcpyHostToDevice, c->io_in));
      CUDA_TRY(cudaMemcpyAsync(base + c->slay.stage_k, (const char*)k_host + t * kb, kb, cudaMemcpyHostToDevice, c->io_in));
      CUDA_TRY(cudaMemcpyAsync(base + c->slay.stage_v, (const char*)v_host + t * kb, kb, cudaMemcpyHostToDevice, c->io_in));
    }
    CUDA_TRY(cudaEventRecord(c->io_in_done[par], c->io_in));
    CUDA_TRY(cudaStreamWaitEvent(s, c->io_in_done[par], 0));
    if (b >= 2) CUDA_TRY(cudaStreamWaitEvent(s, c->io_out_done[par], 0));
    for (int i = 0; i < cnt; ++i) {
      char* base = set_base(i);
      d2o_status why = D2O_OK;
      cudaError_t e = launch_decode(c, l0, l1, base + c->slay.stage_q, base + c->slay.stage_k, base + c->slay.stage_v,
                                    base + c->slay.stage_out, s, &why, i > 0, i + 1 < cnt);
      if (why != D2O_OK || e != cudaSuccess) {
        (void)cudaStreamSynchronize(c->io_in); (void)cudaStreamSynchronize(c->io_out); (void)cudaStreamSynchronize(s);
        return why != D2O_OK ? why : cuda_fail(e, "launch_decode");
      }
      for (int l = l0; l < l1; ++l) c->layer_steps[l] += 1;
    }
    CUDA_TRY(cudaEventRecord(c->io_step_done[par], s));
    CUDA_TRY(cudaStreamWaitEvent(c->io_out, c->io_step_done[par], 0));
    for (int i = 0; i < cnt; ++i)
      CUDA_TRY(cudaMemcpyAsync((char*)out_host + (size_t)(t0 + i) * qb, set_base(i) + c->slay.stage_out, qb,
                               cudaMemcpyDeviceToHost, c->io_out));
    CUDA_TRY(cudaEventRecord(c->io_out_done[par], c->io_out));
  }
  // the caller's stream ends behind the last copies back; then wait for all of it
  for (int i = 0; i < (n_blocks > 1 ? 2 : 1); ++i) CUDA_TRY(cudaStreamWaitEvent(s, c->io_out_done[(n_blocks - 1 - i) & 1], 0));
  CUDA_TRY(cudaStreamSynchronize(s));
  return D2O_OK;
}

extern "C" d2o_status d2o_full_decode_step(int32_t dtype, int32_t d_head, int32_t n_slices, int32_t group,
                                           int32_t capacity, int32_t len, void* k_cache, void* v_cache,
                                           const void* q, const void* k, const void* v, void* out, void* stream) {
  if (dtype != D2O_F32 && dtype != D2O_F16 && dtype != D2O_BF16) return D2O_ERR_UNSUPPORTED;
  if (d_head != 64 && d_head != 128) return D2O_ERR_UNSUPPORTED;
  if (group != 1 && group != 2 && group != 4 && group != 8) return D2O_ERR_UNSUPPORTED;
  if (n_slices < 1 || capacity < 1 || len < 0 || len >= capacity) return D2O_ERR_INVALID_ARG;
  if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
    return D2O_ERR_INVALID_ARG;
  d2o_status why = D2O_OK;
  cudaError_t e = launch_full_decode(dtype, d_head, n_slices, group, capacity, len, k_cache, v_cache, q, k, v, out,
                                     (cudaStream_t)stream, &why);
  if (why != D2O_OK) return why;
  if (e != cudaSuccess) return cuda_fail(e, "launch_full_decode");
  return D2O_OK;
}

extern "C" d2o_status d2o_get_view(d2o_ctx* c, int32_t layer, d2o_view* v) {
  if (!c || !v || layer < 0 || layer >= c->cfg.n_layers) return D2O_ERR_INVALID_ARG;
  const d2o_config& g = c->cfg;
  const size_t per_layer = (size_t)g.batch * g.n_q_heads * g.prompt_len;
  v->colsum = (const float*)(c->state + c->lay.colsum) + per_layer * layer;
  v->density = (const double*)(c->state + c->lay.density);
  v->budgets = (const int32_t*)(c->state + c->lay.budgets);
  v->windows = (const int32_t*)(c->state + c->lay.windows);
  v->row_off = (const int64_t*)(c->state + c->lay.row_off);
  v->k_cache = c->state + c->lay.kpool;
  v->v_cache = c->state + c->lay.vpool;
  v->pos = (int32_t*)(c->state + c->lay.pos);
  v->score = (float*)(c->state + c->lay.score);
  v->rnorm = (float*)(c->state + c->lay.rnorm);
  v->len = (int32_t*)(c->state + c->lay.len);
  v->tau = (float*)(c->state + c->lay.tau);
  v->evict_idx = (const int32_t*)(c->scratch + c->slay.evict_idx);
  v->evict_mx = (const float*)(c->scratch + c->slay.evict_mx);
  v->evict_nn = (const int32_t*)(c->scratch + c->slay.evict_nn);
  v->pool_rows = c->pool_rows;
  return D2O_OK;
}

extern "C" d2o_status d2o_get_stats(d2o_ctx* c, d2o_stats* out, void* stream) {
  if (!c || !out) return D2O_ERR_INVALID_ARG;
  uint64_t cnt[kNumCounters];
  uint32_t word[4];
  cudaStream_t s = (cudaStream_t)stream;
  CUDA_TRY(cudaMemcpyAsync(cnt, c->state + c->lay.counters, sizeof(cnt), cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaMemcpyAsync(word, c->state + c->lay.status, sizeof(word), cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaStreamSynchronize(s));
  out->decode_steps = cnt[kCntDecodeSteps];
  out->evictions = cnt[kCntEvictions];
  out->merges = cnt[kCntMerges];
  out->discards = cnt[kCntDiscards];
  out->prefill_evicted = cnt[kCntPrefillEvicted];
  out->prefill_merged = cnt[kCntPrefillMerged];
  out->error_word = word[0];
  out->error_detail = word[1];
  out->decode_launches = c->decode_launches;
  out->guess_misses = cnt[kCntGuessMisses];
  return D2O_OK;
}

extern "C" d2o_status d2o_set_tuning(d2o_ctx* c, int32_t decode_stages, int32_t decode_l2_hints,
                                     int32_t similarity_path, int32_t stats_path, int32_t decode_warps,
                                     int32_t decode_smem_rows, int32_t decode_long_pairs) {
  if (!c) return D2O_ERR_INVALID_ARG;
  if (decode_stages < 0 || decode_stages > 12) return D2O_ERR_INVALID_ARG;
  if (decode_l2_hints < 0 || decode_l2_hints > 1) return D2O_ERR_INVALID_ARG;
  if (similarity_path < 0 || similarity_path > 1 || stats_path < 0 || stats_path > 1) return D2O_ERR_INVALID_ARG;
  c->decode_stages = decode_stages;
  c->decode_l2_hints = decode_l2_hints;
  c->similarity_path = similarity_path;
  if (decode_warps != 0 && decode_warps != 4 && decode_warps != 8 && decode_warps != 16) return D2O_ERR_INVALID_ARG;
  if (decode_smem_rows != 0 && decode_smem_rows < 8) return D2O_ERR_INVALID_ARG;
  c->stats_path = stats_path;
  c->decode_warps = decode_warps;
  c->decode_smem_rows = decode_smem_rows;
  c->decode_long_pairs = decode_long_pairs;
  return D2O_OK;
}

extern "C" d2o_status d2o_set_fault_injection(d2o_ctx* c, int32_t wait_limit_us, int32_t producer_stop_stage) {
  if (!c || wait_limit_us < 0 || producer_stop_stage < -1) return D2O_ERR_INVALID_ARG;
  c->wait_limit_us = wait_limit_us;
  c->producer_stop_stage = producer_stop_stage;
  return D2O_OK;
}

extern "C" d2o_status d2o_set_prompt_lens(d2o_ctx* c, const int32_t* lens_host, void* stream) {
  if (!c || !lens_host) return D2O_ERR_INVALID_ARG;
  const d2o_config& g = c->cfg;
  for (int l = 0; l < g.n_layers; ++l)
    if (c->layer_fed[l]) return D2O_ERR_STATE;                 // the lengths belong to the prompt that is about to be fed
  for (int b = 0; b < g.batch; ++b) {
    const int P = lens_host[b];
    if (P < 1 || P > g.prompt_len) return D2O_ERR_INVALID_ARG;
    // the same conditions d2o_create checks for prompt_len, for this sequence
    const int maxb = g.max_budget > 0 ? g.max_budget : P;
    if (maxb > P + g.max_new_tokens || g.min_budget > maxb) return D2O_ERR_INVALID_ARG;
    const double units = g.budget_rule == 1 ? (double)g.n_layers * g.n_kv_heads : (double)g.n_layers;
    const double tot = floor((double)g.rho * units * (double)P + 0.5);
    if (g.budget_rule != 2 && (tot < units * g.min_budget || tot > units * maxb)) return D2O_ERR_INVALID_ARG;
  }
  memcpy(c->h_plen, lens_host, (size_t)g.batch * 4);
  CUDA_TRY(cudaMemcpyAsync(c->state + c->lay.plen, c->h_plen, (size_t)g.batch * 4, cudaMemcpyHostToDevice,
                           (cudaStream_t)stream));
  CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));      // h_plen may change again before the copy would run
  return D2O_OK;
}
