// Shared device/host helpers of the D2O library: element-type traits, 16-byte vector access,
// warp reductions, the context object and the launcher prototypes.  Nothing in here is shared
// with the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/d2o.h"

namespace d2o {

constexpr float kEuler = 2.718281828459045f;   // weight of a conserved token: exp(self-similarity 1), Eq. 12
constexpr float kLog2e = 1.4426950408889634f;

// ----------------------------------------------------------------------------- element traits
template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kPerVec = 4;            // elements per 16-byte vector
  __device__ static __forceinline__ void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static __forceinline__ uint4 pack(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
  }
  __device__ static __forceinline__ float to_float(float x) { return x; }
  __device__ static __forceinline__ float from_float(float x) { return x; }
};
template <> struct Elem<__half> {
  static constexpr int kPerVec = 8;
  __device__ static __forceinline__ void unpack(const uint4& v, float* f) {
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 t = __half22float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
  }
  __device__ static __forceinline__ uint4 pack(const float* f) {
    uint4 v; __half2* h = reinterpret_cast<__half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2half2_rn(f[2 * i], f[2 * i + 1]);
    return v;
  }
  __device__ static __forceinline__ float to_float(__half x) { return __half2float(x); }
  __device__ static __forceinline__ __half from_float(float x) { return __float2half_rn(x); }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  __device__ static __forceinline__ void unpack(const uint4& v, float* f) {
    // bf16 -> f32 is a 16-bit shift
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
  }
  __device__ static __forceinline__ uint4 pack(const float* f) {
    uint4 v; __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    return v;
  }
  __device__ static __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
  __device__ static __forceinline__ __nv_bfloat16 from_float(float x) { return __float2bfloat16_rn(x); }
};

__device__ __forceinline__ uint4 ld_global_v4(const void* p) {
  return *reinterpret_cast<const uint4*>(p);
}
// streaming load: data that is read once per launch should not displace reusable lines in L1
// (plain coherent load: the cache rows are also written later in the same launch)
__device__ __forceinline__ uint4 ld_stream_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// ----------------------------------------------------------------------------- reductions
template <typename T> __device__ __forceinline__ T warp_sum(T v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ unsigned long long warp_min_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { unsigned long long t = __shfl_xor_sync(0xffffffffu, v, o); v = t < v ? t : v; }
  return v;
}
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { unsigned long long t = __shfl_xor_sync(0xffffffffu, v, o); v = t > v ? t : v; }
  return v;
}
// A row of d_head elements is handled by LPR consecutive lanes (one 16-byte segment each).  Groups of
// one warp may diverge (ragged tails), so their shuffles name only the lanes of the group.
template <int LPR> __device__ __forceinline__ unsigned group_mask() {
  if (LPR >= 32) return 0xffffffffu;
  return ((1u << (LPR & 31)) - 1u) << (((threadIdx.x & 31) / LPR) * LPR);
}
template <int LPR> __device__ __forceinline__ float group_sum(float v, unsigned mask) {
#pragma unroll
  for (int o = LPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(mask, v, o);
  return v;
}
// monotone map float -> uint32 (a < b  <=>  ord(a) < ord(b)), -0 and +0 distinct but adjacent
__device__ __forceinline__ uint32_t float_ord(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ord_float(uint32_t o) {
  uint32_t u = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
  return __uint_as_float(u);
}

// Cache rows of one slice (sequence, layer, KV head) start at a multiple of 8 rows, so that the 4-byte
// per-row arrays (pos, score, rnorm) of a slice start on a 32-byte boundary (bulk copies need 16).
__host__ __device__ __forceinline__ int slice_stride(int S) { return (S + 7) & ~7; }

// index of slice (sequence b, layer, KV head h) in the [B, L, Hkv] tables (budgets, windows, row offsets)
__host__ __device__ __forceinline__ int slice_entry(int b, int layer, int h, int L, int Hkv) { return (b * L + layer) * Hkv + h; }

// device-side anomaly report: first writer wins
__device__ __forceinline__ void report_error(uint32_t* status_word, uint32_t code, uint32_t detail) {
  if (atomicCAS(status_word, 0u, code) == 0u) status_word[1] = detail;
}

// Checked build (-DD2O_CHECKED, libd2o_checked.so): every index that a kernel derives from data (a position read
// from a list, a victim or neighbour row, a cache row computed from the tables) is compared with its range before it
// is used.  A violation records D2O_ERR_STATE with a code naming the check and the access is skipped; nothing traps.
// In the ordinary build the guard is the constant `true`.
#ifdef D2O_CHECKED
#define D2O_GUARD(cond, status_word, code) ((cond) ? true : (d2o::report_error((status_word), D2O_ERR_STATE, (code)), false))
#else
#define D2O_GUARD(cond, status_word, code) true
#endif

// ----------------------------------------------------------------------------- counters
enum Counter { kCntDecodeSteps = 0, kCntEvictions, kCntMerges, kCntDiscards, kCntPrefillEvicted,
               kCntPrefillMerged, kCntGuessMisses, kNumCounters = 8 };

// ----------------------------------------------------------------------------- context
struct Layout {            // byte offsets into `state`
  size_t status, counters, density, budgets, windows, row_off, order, plen, len, tau, steps_done, sim_items, colsum, pos, score, rnorm, kpool, vpool, end;
};
struct ScratchLayout {     // byte offsets into `scratch`
  size_t lse, evict_idx, evict_mx, evict_nn, seg_start, seg_items, seg_tmp, part_key, pl_spill, stage_q, stage_k, stage_v, stage_out, end;
  size_t lse_stride;       // `lse` exists kStatsLanes times, this far apart (d2o_layer_stats_layers)
  size_t stage_stride;     // stage_q .. stage_out exist 2 * kHostBlock times, this far apart (d2o_decode_steps_host)
  size_t lane_stride;      // evict_idx .. part_key are the working set of one layer's compression: kCompressLanes copies, this far apart
};
constexpr int kHostBlock = 4;       // steps per block of d2o_decode_steps_host (two blocks of staging sets)
constexpr int kStatsLanes = 2;      // layers whose column sums d2o_layer_stats_layers computes side by side
constexpr int kCompressLanes = 4;   // layers that d2o_prefill_compress_layers works on side by side

}  // namespace d2o

struct d2o_ctx {
  d2o_config cfg;
  int group;
  int elem_size;
  int max_budget;
  int n_sms;                   // multiprocessors of the device the context was created on
  int64_t total_budget;        // S_tot per sequence = round(rho * L * P)
  int64_t pool_rows;           // B * Hkv * S_tot
  d2o::Layout lay;
  d2o::ScratchLayout slay;
  char* state;
  char* scratch;
  size_t state_bytes, scratch_bytes;
  // host mirrors, valid after d2o_layer_budgets
  bool have_budgets;
  int32_t* h_budgets;          // [B, L, Hkv]
  int32_t* h_windows;          // [B, L, Hkv]
  int64_t* h_row_off;          // [B, L, Hkv]
  int32_t* h_pair_max;         // [B, L] largest cache size over the KV heads of the pair
  int64_t* h_pair_sum;         // [B, L] cache sizes summed over the KV heads of the pair
  uint8_t* layer_fed;          // [L] stats seen
  uint8_t* layer_compressed;   // [L]
  int32_t* layer_steps;        // [L] decode steps taken
  int32_t* h_plen;             // [B] prompt length of every sequence (prompt_len unless d2o_set_prompt_lens was called)
  int32_t* h_sim_count;        // [L] work items of the tensor-core similarity kernel per layer
  int4* h_sim_items;           // host copy of the work lists (device copy in `state`)
  int32_t* h_order;            // [L * B] (layer * B + b) sorted by cache size, largest first (device copy in `state`)
  int decode_stages;           // tuning: stages of the decode kernel's ring, 0 = auto
  int decode_warps;            // tuning: consumer warps per decode CTA (4, 8, 16), 0 = auto
  int decode_smem_rows;        // tuning: rows of a slice with their logits in shared memory, 0 = auto
  mutable uint64_t decode_launches;   // decode kernels launched so far
  int decode_long_pairs;       // tuning: (layer, sequence) pairs in the long-slice launch, 0 = auto, < 0 = never
  int decode_l2_hints;         // tuning: 1 = the decode kernel's copies carry L2 eviction hints
  int similarity_path;         // tuning: 0 = tensor cores for 16-bit keys, 1 = FFMA kernel for every dtype
  int stats_path;              // tuning: 0 = tensor cores for the column sums of 16-bit Q/K, 1 = FFMA kernels
  int wait_limit_us;           // failure-detection tests: limit of a device-side wait in microseconds (0 = one second)
  int producer_stop_stage;     // failure-detection tests: the decode producer issues no copy from this stage on (-1 = never)
  // d2o_prefill_compress_layers: one stream per lane, created with the first call (no device memory involved)
  cudaStream_t lane_stream[d2o::kCompressLanes];
  cudaEvent_t lane_done[d2o::kCompressLanes];
  cudaEvent_t lane_fork;
  bool lanes_ready;
  // d2o_decode_steps_host: a stream for the copies to the device, one for the copies back; created with the first call
  cudaStream_t io_in, io_out;
  cudaEvent_t io_start, io_in_done[2], io_step_done[2], io_out_done[2];
  bool io_ready;
};

namespace d2o {

// launchers (one per .cu file); all return cudaError_t of the launch
cudaError_t launch_layer_stats(const d2o_ctx* c, int layer, const void* Q, const void* K, const float* lse,
                               cudaStream_t st, int lane = 0);
cudaError_t launch_budgets(const double* density, int B, int L, int H, int Hkv, int P, float rho, int min_budget,
                           int max_budget, float gamma, int head_reduce, int budget_rule, int n_sink, int window,
                           float nm_ratio, int32_t* budgets, int32_t* windows, int64_t* row_off, uint32_t* status_word,
                           const int32_t* plen, cudaStream_t st);
cudaError_t launch_prefill_compress(const d2o_ctx* c, int layer, const void* K, const void* V, cudaStream_t st, int lane = 0);
cudaError_t launch_decode(const d2o_ctx* c, int l0, int l1, const void* q, const void* k, const void* v, void* out,
                          cudaStream_t st, d2o_status* why, bool chained = false, bool publish = false);
cudaError_t launch_full_decode(int dtype, int d, int n_slices, int group, int capacity, int len, void* kc, void* vc,
                               const void* q, const void* k, const void* v, void* out, cudaStream_t st,
                               d2o_status* why);

// tensor-core similarity + nearest neighbour for 16-bit keys (d2o_sim_tc.cu); fills evict_mx / evict_nn
cudaError_t launch_similarity_tc(const d2o_ctx* c, int layer, const void* K, int max_S, cudaStream_t st, int lane = 0);
size_t sim_tc_part_key_bytes(const d2o_config* cfg, int max_budget);
size_t sim_tc_max_items(const d2o_config* cfg, int max_budget);
void sim_tc_build_items(const d2o_ctx* c, int n_sms, int4* items, int32_t* count);
// tensor-core column sums of the prompt attention for 16-bit Q/K (d2o_colsum_tc.cu)
bool colsum_tc_supported(const d2o_config* cfg);
cudaError_t launch_colsum_tc(const d2o_ctx* c, const void* Q, const void* K, const float* lse_in, float* colsum,
                             cudaStream_t st, int lane = 0);

// remembers the text of a failed CUDA runtime call for d2o_last_cuda_error(); returns D2O_ERR_CUDA
d2o_status record_cuda_error(cudaError_t e, const char* where);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace d2o
