// Token-level operation at the prompt stage (Section 4.2): eviction (Eq. 7-8), nearest-neighbour
// matching (Eq. 9), the initial threshold (Eq. 10, t = 0) and weighted merging (Eq. 11-12).
//
// Kernels in this file, per layer, one slice = one (sequence, KV head):
//   select_kernel      group-summed scores, block radix select of the Top-N under the order
//                      (score desc, position asc), ordered compaction into retained / evicted
//                      position lists and the retained scores
//   gather_kernel      K_c, V_c and inverse key norms of the retained positions
//   similarity_kernel  cosine of every evicted key with every retained key, row max / arg-max
//                      (generic FFMA version; 16-bit inputs take the tcgen05 kernel when built in)
//   segment_kernel     tau_0 = mean of the row maxima; threshold test; evicted tokens grouped by
//                      their nearest neighbour in ascending position (deterministic lists)
//   merge_kernel       per retained row: (e*k_c + sum exp(u)*k_e) / (e + sum exp(u)), same for V
#include <math.h>

#include "d2o_common.cuh"

namespace d2o {

// ------------------------------------------------------------------------------------ select
constexpr int kSelThreads = 1024;

struct SelectArgs {
  const float* colsum;     // [B, Hq, P] of this layer
  const int32_t* budgets;  // [B, L, Hkv]
  const int32_t* windows;  // [B, L, Hkv]
  const int64_t* row_off;  // [B, L, Hkv]
  int32_t* pos; float* score; float* rnorm;   // pool-wide
  int32_t* len; float* tau;                   // [L, B, Hkv]
  int32_t* steps_done;                        // [L, B, Hkv] decode steps completed on the slice
  int32_t* evict_idx;      // [B, Hkv, P]
  float* keys_spill;       // [B, Hkv, P] group scores when P does not fit in shared memory (may alias evict_mx)
  unsigned long long* counters;
  uint32_t* status;
  const int32_t* plen;     // [B] prompt length of every sequence; P below is the length the tensors are laid out for
  int L, layer, B, Hq, Hkv, G, P, T;
  int keys_in_smem;
  long long pool_rows;     // rows of the cache pool (bounds of the checked build)
  int value_feature;       // 1: the similarity of Eq. 9 is taken on the value rows (ablation), so the norms are theirs
};

__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot, int* total) {
  // exclusive prefix of v over the block (blockDim multiple of 32, <= 1024)
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
  __syncthreads();
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = lane < (int)(blockDim.x >> 5) ? warp_tot[lane] : 0;
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xffffffffu, winc, o); if (lane >= o) winc += t; }
    warp_tot[lane] = winc - w;
    if (lane == 31) *total = winc;
  }
  __syncthreads();
  return inc - v + warp_tot[warp];
}

template <typename T, int D>
__global__ void __launch_bounds__(kSelThreads)
select_kernel(SelectArgs a, const T* __restrict__ K, const T* __restrict__ V, T* __restrict__ kpool,
              T* __restrict__ vpool) {
  extern __shared__ __align__(16) unsigned char sel_smem[];
  __shared__ int hist[256];
  __shared__ int warp_tot[32];
  __shared__ int s_total;
  __shared__ uint32_t s_prefix;
  __shared__ int s_need;
  const int slice = blockIdx.x;                 // b * Hkv + h
  const int b = slice / a.Hkv, h = slice % a.Hkv;
  const int Pmax = a.P;                         // row stride of the per-position arrays
  const int P = a.plen[b];                      // this sequence's prompt length
  const int S = a.budgets[slice_entry(b, a.layer, h, a.L, a.Hkv)];
  const int Tn = a.T < S ? a.T : S;
  const int M = a.windows[slice_entry(b, a.layer, h, a.L, a.Hkv)];
  const int64_t row0 = a.row_off[slice_entry(b, a.layer, h, a.L, a.Hkv)];
  const int sidx = (a.layer * a.B + b) * a.Hkv + h;
  float* keys = a.keys_in_smem ? reinterpret_cast<float*>(sel_smem) : a.keys_spill + (size_t)slice * Pmax;
  // group score: sum over the G query heads of this KV head, fixed order (Eq. 6 case 1)
  const float* cs = a.colsum + ((size_t)b * a.Hq + (size_t)h * a.G) * Pmax;
  for (int j = threadIdx.x; j < P; j += blockDim.x) {
    float t = cs[j];
    for (int g = 1; g < a.G; ++g) t += cs[(size_t)g * Pmax + j];
    keys[j] = t;
  }
  __syncthreads();
  const bool keep_all = S >= P;
  const int lo = Tn, hi = keep_all ? Tn : P - M;   // candidate range [lo, hi)
  const int N = S - Tn - M;
  uint32_t kth = 0; int need_eq = 0;
  if (!keep_all && N > 0) {
    // radix select of the N-th largest key among candidates; scores are >= 0 so the IEEE bit
    // pattern is monotone, float_ord keeps it monotone for any sign
    uint32_t prefix = 0, mask = 0; int need = N;
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
      __syncthreads();
      for (int j = lo + threadIdx.x; j < hi; j += blockDim.x) {
        const uint32_t o = float_ord(keys[j]);
        if ((o & mask) == prefix) atomicAdd(&hist[(o >> shift) & 255], 1);
      }
      __syncthreads();
      if (threadIdx.x == 0) {
        int acc = 0, bin = 255;
        for (; bin > 0; --bin) { if (acc + hist[bin] >= need) break; acc += hist[bin]; }
        s_prefix = prefix | ((uint32_t)bin << shift);
        s_need = need - acc;
      }
      __syncthreads();
      prefix = s_prefix; need = s_need; mask |= 255u << shift;
      __syncthreads();
    }
    kth = prefix; need_eq = need;                 // keep all keys > kth and the first need_eq keys == kth
  }
  // ordered compaction over positions, 1024 at a time
  int n_ret = 0, n_ev = 0, n_eq = 0;
  for (int base = 0; base < P; base += blockDim.x) {
    const int j = base + threadIdx.x;
    int is_eq = 0, keep = 0;
    uint32_t o = 0;
    if (j < P) {
      if (keep_all || j < Tn || j >= P - M) keep = 1;
      else if (N > 0) { o = float_ord(keys[j]); if (o > kth) keep = 1; else if (o == kth) is_eq = 1; }
    }
    const int eq_rank = block_exclusive_scan(is_eq, warp_tot, &s_total);
    const int eq_tot = s_total;
    if (is_eq && n_eq + eq_rank < need_eq) keep = 1;
    const int kr = block_exclusive_scan(keep, warp_tot, &s_total);
    const int keep_tot = s_total;
    if (j < P) {
      if (keep) {
        const int slot = n_ret + kr;
        if (D2O_GUARD(slot < (keep_all ? P : S) && row0 + slot < a.pool_rows, a.status, 0xC4EC0001u)) {
          a.pos[row0 + slot] = j;
          a.score[row0 + slot] = keys[j];
        }
      } else {
        const int at = n_ev + (threadIdx.x - kr);
        if (D2O_GUARD(at >= 0 && at < P, a.status, 0xC4EC0002u)) a.evict_idx[(size_t)slice * Pmax + at] = j;
      }
    }
    const int valid = min((int)blockDim.x, P - base);
    n_ret += keep_tot; n_ev += valid - keep_tot; n_eq += eq_tot;
    __syncthreads();
  }
  const int n_keep = keep_all ? P : S;
  if (threadIdx.x == 0) {
    a.len[sidx] = n_keep;
    a.steps_done[sidx] = 0;
    a.tau[sidx] = 0.f;
    if (n_ret != n_keep) report_error(a.status, D2O_ERR_STATE, 0x5E000000u | (uint32_t)slice);
    atomicAdd(&a.counters[kCntPrefillEvicted], (unsigned long long)(P - n_keep));
  }
}

// Gather of K_c, V_c and 1/|k| for the positions select_kernel wrote: one row per LPR-lane group, 64 rows per CTA
// (a kernel of its own so that a single sequence still fills the GPU).
template <typename T, int D>
__global__ void __launch_bounds__(256)
gather_kernel(SelectArgs a, const T* __restrict__ K, const T* __restrict__ V, T* __restrict__ kpool,
              T* __restrict__ vpool) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int LPR = D / EPV;                   // lanes per row
  const int slice = blockIdx.y;
  const int b = slice / a.Hkv, h = slice % a.Hkv;
  const int P = a.plen[b];
  const int S = a.budgets[slice_entry(b, a.layer, h, a.L, a.Hkv)];
  const int n_keep = S >= P ? P : S;
  const int64_t row0 = a.row_off[slice_entry(b, a.layer, h, a.L, a.Hkv)];
  const int grp = threadIdx.x / LPR, lig = threadIdx.x % LPR;
  const T* Ks = K + (size_t)slice * a.P * D;
  const T* Vs = V + (size_t)slice * a.P * D;
  const int r1 = min(n_keep, ((int)blockIdx.x + 1) * 64);
  for (int r = blockIdx.x * 64 + grp; r < r1; r += blockDim.x / LPR) {
    const int j = a.pos[row0 + r];
    if (!D2O_GUARD(j >= 0 && j < P && row0 + r < a.pool_rows, a.status, 0xC4EC0003u)) continue;
    const uint4 kv = ld_global_v4(Ks + (size_t)j * D + lig * EPV);
    const uint4 vv = ld_global_v4(Vs + (size_t)j * D + lig * EPV);
    *reinterpret_cast<uint4*>(kpool + (row0 + r) * D + lig * EPV) = kv;
    *reinterpret_cast<uint4*>(vpool + (row0 + r) * D + lig * EPV) = vv;
    float f[EPV]; Elem<T>::unpack(a.value_feature ? vv : kv, f);
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < EPV; ++i) ss = fmaf(f[i], f[i], ss);
    ss = group_sum<LPR>(ss, group_mask<LPR>());
    if (lig == 0) a.rnorm[row0 + r] = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
  }
}

// ------------------------------------------------------------------------------------ similarity (generic)
constexpr int kSimTile = 64;
constexpr int kSimThreads = 256;

struct SimArgs {
  const int32_t* budgets; const int64_t* row_off;
  const int32_t* evict_idx; float* evict_mx; int32_t* evict_nn;
  const float* rnorm; const int32_t* pos;
  uint32_t* status;
  const int32_t* plen;
  int L, layer, Hkv, P;
};

template <typename T, int D>
__global__ void __launch_bounds__(kSimThreads)
similarity_kernel(SimArgs a, const T* __restrict__ K, const T* __restrict__ kpool) {
  extern __shared__ __align__(16) float sim_smem[];
  float* et = sim_smem;                     // [D][64] evicted tile, transposed
  float* ct = et + D * kSimTile;            // [D][64] retained tile, transposed
  float* ern = ct + D * kSimTile;           // [64] inverse norms of the evicted rows
  float* crn = ern + kSimTile;              // [64] inverse norms of the retained rows
  const int slice = blockIdx.y;
  const int b = slice / a.Hkv, h = slice % a.Hkv;
  const int S = a.budgets[slice_entry(b, a.layer, h, a.L, a.Hkv)];
  const int Le = a.plen[b] - S;
  const int i0 = blockIdx.x * kSimTile;
  if (Le <= 0 || i0 >= Le) return;
  const int64_t row0 = a.row_off[slice_entry(b, a.layer, h, a.L, a.Hkv)];
  const T* Ks = K + (size_t)slice * a.P * D;
  const int32_t* ev = a.evict_idx + (size_t)slice * a.P;
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int VPR = D / EPV;
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
  {  // evicted tile: gather rows by index, transposed, plus inverse norms
    const int r = threadIdx.x % kSimTile;
    bool ok = i0 + r < Le;
    const int j = ok ? ev[i0 + r] : 0;
    if (ok && !D2O_GUARD(j >= 0 && j < a.plen[b], a.status, 0xC4EC0004u)) ok = false;
    float ss = 0.f;
    for (int vi = threadIdx.x / kSimTile; vi < VPR; vi += kSimThreads / kSimTile) {
      float f[EPV];
      if (ok) { uint4 v = ld_global_v4(Ks + (size_t)j * D + vi * EPV); Elem<T>::unpack(v, f); }
      else {
#pragma unroll
        for (int i = 0; i < EPV; ++i) f[i] = 0.f;
      }
#pragma unroll
      for (int i = 0; i < EPV; ++i) { et[(vi * EPV + i) * kSimTile + r] = f[i]; ss = fmaf(f[i], f[i], ss); }
    }
    // 4 threads (tid/64 = 0..3) share a row: each partial norm goes to its own cell of ct[]
    // (not yet in use) and is combined in a fixed order
    ct[(threadIdx.x / kSimTile) * kSimTile + r] = ss;
    __syncthreads();
    if (threadIdx.x < kSimTile) {
      const float t = (ct[r] + ct[kSimTile + r]) + (ct[2 * kSimTile + r] + ct[3 * kSimTile + r]);
      ern[r] = t > 0.f ? 1.0f / sqrtf(t) : 0.f;
    }
    __syncthreads();
  }
  float best[4]; int bidx[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) { best[r] = -INFINITY; bidx[r] = 0x7fffffff; }
  for (int c0 = 0; c0 < S; c0 += kSimTile) {
    __syncthreads();
    {
      const int r = threadIdx.x % kSimTile;
      const bool ok = c0 + r < S;
      for (int vi = threadIdx.x / kSimTile; vi < VPR; vi += kSimThreads / kSimTile) {
        float f[EPV];
        if (ok) { uint4 v = ld_global_v4(kpool + (row0 + c0 + r) * D + vi * EPV); Elem<T>::unpack(v, f); }
        else {
#pragma unroll
          for (int i = 0; i < EPV; ++i) f[i] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < EPV; ++i) ct[(vi * EPV + i) * kSimTile + r] = f[i];
      }
      if (threadIdx.x < kSimTile) crn[r] = ok ? a.rnorm[row0 + c0 + r] : 0.f;
    }
    __syncthreads();
    float s[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) s[r][c] = 0.f;
#pragma unroll 8
    for (int k = 0; k < D; ++k) {
      const float4 av = *reinterpret_cast<const float4*>(et + k * kSimTile + ty * 4);
      const float4 bv = *reinterpret_cast<const float4*>(ct + k * kSimTile + tx * 4);
      const float aa[4] = {av.x, av.y, av.z, av.w};
      const float bb[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) s[r][c] = fmaf(aa[r], bb[c], s[r][c]);
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const float er = ern[ty * 4 + r];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int col = c0 + tx * 4 + c;
        if (col < S) {
          const float u = s[r][c] * er * crn[tx * 4 + c];
          if (u > best[r]) { best[r] = u; bidx[r] = col; }       // ascending col: first maximum wins
        }
      }
    }
  }
  // combine the 16 threads (tx) of a row: max u, ties -> lowest slot
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    // -0 (a zero-norm row) counts as +0, so that equal similarities tie
    unsigned long long key = ((unsigned long long)float_ord(__fadd_rn(best[r], 0.f)) << 32) | (uint32_t)(0x7fffffff - bidx[r]);
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
      const unsigned long long t = __shfl_xor_sync(0xffffffffu, key, o);
      key = t > key ? t : key;
    }
    const int i = i0 + ty * 4 + r;
    if (tx == 0 && i < Le) {
      // a row whose similarities are all NaN keeps the initial key: maximum -inf, neighbour 0, never merged
      const int slot = 0x7fffffff - (int)(uint32_t)(key & 0xffffffffu);
      const bool found = (unsigned)slot < (unsigned)S;
      a.evict_mx[(size_t)slice * a.P + i] = found ? ord_float((uint32_t)(key >> 32)) : -INFINITY;
      a.evict_nn[(size_t)slice * a.P + i] = found ? slot : 0;
    }
  }
}

// ------------------------------------------------------------------------------------ tau_0 + segments
struct SegArgs {
  const int32_t* budgets;
  const float* evict_mx; const int32_t* evict_nn;
  int32_t* seg_start; int32_t* seg_items; int32_t* seg_tmp; float* tau;
  unsigned long long* counters;
  uint32_t* status;
  const int32_t* plen;
  int L, layer, B, Hkv, P, seg_stride;
  float tau_override;
};

__global__ void __launch_bounds__(1024)
segment_kernel(SegArgs a) {
  extern __shared__ __align__(16) int seg_smem[];       // [max(S + 1, 32 * 64)] counts / cursors, then radix histograms
  __shared__ double part[32];
  __shared__ float s_thr;
  __shared__ int warp_tot[32];
  __shared__ int s_total;
  const int slice = blockIdx.x;
  const int b = slice / a.Hkv, h = slice % a.Hkv;
  const int S = a.budgets[slice_entry(b, a.layer, h, a.L, a.Hkv)];
  const int Le = a.plen[b] - S;
  const int sidx = (a.layer * a.B + b) * a.Hkv + h;
  const float* mx = a.evict_mx + (size_t)slice * a.P;
  const int32_t* nn = a.evict_nn + (size_t)slice * a.P;
  int32_t* start = a.seg_start + (size_t)slice * a.seg_stride;
  int32_t* items = a.seg_items + (size_t)slice * a.P;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (Le <= 0) {
    for (int j = threadIdx.x; j <= S && j < a.seg_stride; j += blockDim.x) start[j] = 0;
    if (threadIdx.x == 0) a.tau[sidx] = 0.f;
    return;
  }
  // tau_0 = (1/Le) sum_i mx_i   (Eq. 10, t = 0); fixed reduction tree, double accumulation
  double t = 0.0;
  for (int i = threadIdx.x; i < Le; i += blockDim.x) t += (double)mx[i];
  t = warp_sum(t);
  if (lane == 0) part[warp] = t;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += part[w];
    const float tau0 = (float)(s / (double)Le);
    a.tau[sidx] = tau0;
    s_thr = isnan(a.tau_override) ? tau0 : a.tau_override;
  }
  for (int j = threadIdx.x; j <= S; j += blockDim.x) seg_smem[j] = 0;
  __syncthreads();
  const float thr = s_thr;
  // An evicted token is merged iff its best similarity reaches the threshold.  A row without a finite maximum or
  // with a neighbour outside the slice (non-finite keys) is never merged; it is reported once per slice.
  auto merges = [&](int i) { return mx[i] >= thr && mx[i] > -INFINITY && (unsigned)nn[i] < (unsigned)S; };
  bool bad_row = false;
  // how many evicted tokens pass the threshold for each retained slot (integer counts: order-free)
  for (int i = threadIdx.x; i < Le; i += blockDim.x) {
    if (merges(i)) atomicAdd(&seg_smem[nn[i]], 1);
    else if (!(mx[i] > -INFINITY) || (unsigned)nn[i] >= (unsigned)S) bad_row = true;
  }
  if (bad_row) report_error(a.status, D2O_ERR_STATE, 0x5E600000u | (uint32_t)(slice & 0xfffff));
  __syncthreads();
  // exclusive scan of the counts -> segment starts
  int run = 0;
  for (int base = 0; base <= S; base += blockDim.x) {
    const int j = base + threadIdx.x;
    const int c = j < S ? seg_smem[j] : 0;
    const int ex = block_exclusive_scan(c, warp_tot, &s_total);
    if (j <= S) { start[j] = run + ex; }
    __syncthreads();
    if (j < S) seg_smem[j] = run + ex;                   // becomes the fill cursor
    run += s_total;
    __syncthreads();
  }
  if (threadIdx.x == 0) atomicAdd(&a.counters[kCntPrefillMerged], (unsigned long long)run);
  // Ordered fill: the passing evicted tokens sorted by (neighbour, index), so that every segment lists its tokens in
  // ascending position.  Stable least-significant-digit radix sort on the neighbour slot, 6 bits per pass; each
  // warp owns a contiguous chunk of the source, counts its digits, and after a scan over (digit, warp) scatters its
  // chunk in order (lanes with the same digit are ranked with match_any).
  if (run == 0) return;
  int* hist = reinterpret_cast<int*>(seg_smem);         // [32 warps][64 digits]; the cursors are not needed any more
  int32_t* tmp = a.seg_tmp + (size_t)slice * a.P;
  int bits = 0;
  while ((S >> bits) != 0) ++bits;                      // slots are < S
  const int passes = (bits + 5) / 6;
  const int n_warps = (int)(blockDim.x >> 5);
  for (int p = 0; p < passes; ++p) {
    // the last pass must land in `items`
    int32_t* dst = ((passes - 1 - p) & 1) ? tmp : items;
    const int32_t* src = dst == items ? tmp : items;    // unused in pass 0 (the source is the index range itself)
    const int n_src = p == 0 ? Le : run;
    const int chunk = (((n_src + n_warps - 1) / n_warps) + 31) & ~31;
    const int c0 = warp * chunk, c1 = min(n_src, c0 + chunk);
    const int shift = 6 * p;
    __syncthreads();
    for (int i = threadIdx.x; i < n_warps * 64; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    for (int base = c0; base < c1; base += 32) {
      const int k = base + lane;
      int item = -1;
      if (k < c1) {
        if (p == 0) { if (merges(k)) item = k; }
        else item = src[k];
      }
      if (item >= 0) atomicAdd(&hist[warp * 64 + ((nn[item] >> shift) & 63)], 1);
    }
    __syncthreads();
    // exclusive scan in (digit, warp) order: 64 * n_warps entries, two per thread
    {
      const int e0 = 2 * threadIdx.x, e1 = e0 + 1;
      const int total_e = 64 * n_warps;
      const int v0 = e0 < total_e ? hist[(e0 % n_warps) * 64 + e0 / n_warps] : 0;
      const int v1 = e1 < total_e ? hist[(e1 % n_warps) * 64 + e1 / n_warps] : 0;
      const int ex = block_exclusive_scan(v0 + v1, warp_tot, &s_total);
      if (e0 < total_e) hist[(e0 % n_warps) * 64 + e0 / n_warps] = ex;
      if (e1 < total_e) hist[(e1 % n_warps) * 64 + e1 / n_warps] = ex + v0;
    }
    __syncthreads();
    for (int base = c0; base < c1; base += 32) {
      const int k = base + lane;
      int item = -1;
      if (k < c1) {
        if (p == 0) { if (merges(k)) item = k; }
        else item = src[k];
      }
      const int dgt = item >= 0 ? ((nn[item] >> shift) & 63) : 64 + lane;   // distinct dummies for idle lanes
      const unsigned peers = __match_any_sync(0xffffffffu, dgt);
      if (item >= 0) {
        const int rank = __popc(peers & ((1u << lane) - 1u));
        const int cur = hist[warp * 64 + dgt];
        dst[cur + rank] = item;
        __syncwarp(peers);
        if (rank == 0) hist[warp * 64 + dgt] = cur + __popc(peers);
      }
      __syncwarp();
    }
    __threadfence_block();
  }
}

// ------------------------------------------------------------------------------------ merge
struct MergeArgs {
  const int32_t* budgets; const int64_t* row_off;
  const int32_t* evict_idx; const float* evict_mx;
  const int32_t* seg_start; const int32_t* seg_items;
  float* rnorm;
  const int32_t* plen;
  int L, layer, Hkv, P, seg_stride;
  uint32_t* status;
  int average;             // 1: average merge (every token of a merge weighs the same) instead of Eq. 12
  int value_feature;       // 1: the cached inverse norms belong to the value rows
};

constexpr int kMergeFlight = 4;     // merged tokens whose rows a row group has in flight

template <typename T, int D>
__global__ void __launch_bounds__(256)
merge_kernel(MergeArgs a, const T* __restrict__ K, const T* __restrict__ V, T* __restrict__ kpool,
             T* __restrict__ vpool) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int LPR = D / EPV;
  const int slice = blockIdx.y;
  const int b = slice / a.Hkv, h = slice % a.Hkv;
  const int S = a.budgets[slice_entry(b, a.layer, h, a.L, a.Hkv)];
  const int Le = a.plen[b] - S;
  if (Le <= 0) return;
  const int grp = threadIdx.x / LPR, lig = threadIdx.x % LPR;
  const int j = blockIdx.x * (blockDim.x / LPR) + grp;
  if (j >= S) return;
  const int32_t* start = a.seg_start + (size_t)slice * a.seg_stride;
  const int s0 = start[j], s1 = start[j + 1];
  if (s1 == s0) return;                              // nothing merged: the row stays bit-identical
  if (!D2O_GUARD(s0 >= 0 && s0 < s1 && s1 <= Le, a.status, 0xC4EC0007u)) return;
  const int64_t row = a.row_off[slice_entry(b, a.layer, h, a.L, a.Hkv)] + j;
  const int32_t* items = a.seg_items + (size_t)slice * a.P;
  const int32_t* ev = a.evict_idx + (size_t)slice * a.P;
  const float* mx = a.evict_mx + (size_t)slice * a.P;
  const T* Ks = K + (size_t)slice * a.P * D;
  const T* Vs = V + (size_t)slice * a.P * D;
  float ka[EPV], va[EPV], f[EPV];
  Elem<T>::unpack(ld_global_v4(kpool + row * D + lig * EPV), f);
  const float own = a.average ? 1.0f : kEuler;       // weight of the retained token itself: e^{self-similarity}, or 1
#pragma unroll
  for (int i = 0; i < EPV; ++i) ka[i] = own * f[i];
  Elem<T>::unpack(ld_global_v4(vpool + row * D + lig * EPV), f);
#pragma unroll
  for (int i = 0; i < EPV; ++i) va[i] = own * f[i];
  float den = own;
  // The lanes of the row first fetch the list entries of up to LPR merged tokens side by side (entry -> similarity and
  // prompt position), then the rows are added in list order, four tokens' key and value rows in flight at a time: the
  // chain entry -> position -> row is three dependent loads per token otherwise, and a retained token that is the
  // neighbour of hundreds of evicted ones is the launch's critical path.
  const unsigned gm = group_mask<LPR>();
  for (int s = s0; s < s1; s += LPR) {
    const int cnt = min(LPR, s1 - s);
    float my_w = 0.f; int my_pj = 0;
    if (lig < cnt) {
      const int i = items[s + lig];
      if (D2O_GUARD(i >= 0 && i < Le, a.status, 0xC4EC0005u)) {
        const int pj = ev[i];
        if (D2O_GUARD(pj >= 0 && pj < a.plen[b], a.status, 0xC4EC0006u)) { my_pj = pj; my_w = a.average ? 1.0f : expf(mx[i]); }
      }
    }
    for (int t = 0; t < cnt; t += kMergeFlight) {
      float w[kMergeFlight]; uint4 kr[kMergeFlight], vr[kMergeFlight];
#pragma unroll
      for (int u = 0; u < kMergeFlight; ++u) {
        const int tu = t + u < cnt ? t + u : t;              // past the list: the first row once more, never added
        w[u] = __shfl_sync(gm, my_w, tu, LPR);
        const int pu = __shfl_sync(gm, my_pj, tu, LPR);
        kr[u] = ld_global_v4(Ks + (size_t)pu * D + lig * EPV);
        vr[u] = ld_global_v4(Vs + (size_t)pu * D + lig * EPV);
      }
#pragma unroll
      for (int u = 0; u < kMergeFlight; ++u) {
        if (t + u < cnt) {                                   // list order; a token whose check failed has weight 0: its terms are +0
          den += w[u];
          Elem<T>::unpack(kr[u], f);
#pragma unroll
          for (int e = 0; e < EPV; ++e) ka[e] = fmaf(w[u], f[e], ka[e]);
          Elem<T>::unpack(vr[u], f);
#pragma unroll
          for (int e = 0; e < EPV; ++e) va[e] = fmaf(w[u], f[e], va[e]);
        }
      }
    }
  }
  const float inv = 1.0f / den;
#pragma unroll
  for (int e = 0; e < EPV; ++e) { ka[e] = ka[e] * inv; va[e] = va[e] * inv; }
  const uint4 kv = Elem<T>::pack(ka), vv = Elem<T>::pack(va);
  *reinterpret_cast<uint4*>(kpool + row * D + lig * EPV) = kv;
  *reinterpret_cast<uint4*>(vpool + row * D + lig * EPV) = vv;
  Elem<T>::unpack(a.value_feature ? vv : kv, f);     // the norm of what is actually stored
  float ss = 0.f;
#pragma unroll
  for (int e = 0; e < EPV; ++e) ss = fmaf(f[e], f[e], ss);
  ss = group_sum<LPR>(ss, group_mask<LPR>());
  if (lig == 0) a.rnorm[row] = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
}

// ------------------------------------------------------------------------------------ launcher
template <typename T, int D>
static cudaError_t run_prefill(const d2o_ctx* c, int layer, const void* K, const void* V, cudaStream_t st, int lane) {
  const d2o_config& g = c->cfg;
  const int B = g.batch, Hkv = g.n_kv_heads, P = g.prompt_len, L = g.n_layers;
  const int n_slices = B * Hkv;
  char* S = c->state; char* X = c->scratch + (size_t)lane * c->slay.lane_stride;   // only the lane's arrays are used below
  T* kpool = (T*)(S + c->lay.kpool);
  T* vpool = (T*)(S + c->lay.vpool);
  int maxS = 0;
  for (int b = 0; b < B; ++b) maxS = max(maxS, c->h_pair_max[b * L + layer]);
  const int seg_stride = c->max_budget + 2;

  SelectArgs sa;
  sa.colsum = (const float*)(S + c->lay.colsum) + (size_t)layer * B * g.n_q_heads * P;
  sa.budgets = (const int32_t*)(S + c->lay.budgets);
  sa.windows = (const int32_t*)(S + c->lay.windows);
  sa.row_off = (const int64_t*)(S + c->lay.row_off);
  sa.pos = (int32_t*)(S + c->lay.pos); sa.score = (float*)(S + c->lay.score); sa.rnorm = (float*)(S + c->lay.rnorm);
  sa.len = (int32_t*)(S + c->lay.len); sa.tau = (float*)(S + c->lay.tau);
  sa.steps_done = (int32_t*)(S + c->lay.steps_done);
  sa.evict_idx = (int32_t*)(X + c->slay.evict_idx);
  sa.keys_spill = (float*)(X + c->slay.evict_mx);
  sa.counters = (unsigned long long*)(S + c->lay.counters);
  sa.status = (uint32_t*)(S + c->lay.status);
  sa.plen = (const int32_t*)(S + c->lay.plen);
  sa.L = L; sa.layer = layer; sa.B = B; sa.Hq = g.n_q_heads; sa.Hkv = Hkv; sa.G = c->group; sa.P = P; sa.T = g.n_sink;
  const size_t key_bytes = (size_t)P * sizeof(float);
  sa.keys_in_smem = key_bytes <= 200 * 1024;
  sa.pool_rows = c->pool_rows;
  sa.value_feature = g.sim_feature;
  const size_t sel_sm = sa.keys_in_smem ? key_bytes : 0;
  cudaError_t e = cudaFuncSetAttribute(select_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)(sel_sm > 48 * 1024 ? sel_sm : 48 * 1024));
  if (e != cudaSuccess) return e;
  select_kernel<T, D><<<n_slices, kSelThreads, sel_sm, st>>>(sa, (const T*)K, (const T*)V, kpool, vpool);
  {
    const int keep_max = min(maxS, P);
    dim3 ggrid((unsigned)((keep_max + 63) / 64), (unsigned)n_slices);
    gather_kernel<T, D><<<ggrid, 256, 0, st>>>(sa, (const T*)K, (const T*)V, kpool, vpool);
  }

  int maxLe = 0;                                 // most evicted rows of any slice of this layer
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < Hkv; ++h) maxLe = max(maxLe, c->h_plen[b] - c->h_budgets[(b * L + layer) * Hkv + h]);
  if (maxLe <= 0) return cudaGetLastError();

  SimArgs ma;
  ma.budgets = sa.budgets; ma.row_off = sa.row_off;
  ma.evict_idx = sa.evict_idx; ma.evict_mx = (float*)(X + c->slay.evict_mx); ma.evict_nn = (int32_t*)(X + c->slay.evict_nn);
  ma.rnorm = sa.rnorm; ma.pos = sa.pos; ma.status = sa.status; ma.plen = sa.plen; ma.L = L; ma.layer = layer; ma.Hkv = Hkv; ma.P = P;
  const size_t sim_sm = ((size_t)2 * D * kSimTile + 2 * kSimTile) * sizeof(float);
  e = cudaFuncSetAttribute(similarity_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sim_sm);
  if (e != cudaSuccess) return e;
  // rows the similarity is computed on: the keys (Eq. 9), or the values (ablation "Feature choice")
  const void* feat = g.sim_feature ? V : K;
  const T* feat_pool = g.sim_feature ? vpool : kpool;
  if (sizeof(T) == 2 && c->similarity_path == 0) {
    e = launch_similarity_tc(c, layer, feat, maxS, st, lane);
    if (e != cudaSuccess) return e;
  } else {
    dim3 sgrid((maxLe + kSimTile - 1) / kSimTile, n_slices);
    similarity_kernel<T, D><<<sgrid, kSimThreads, sim_sm, st>>>(ma, (const T*)feat, feat_pool);
  }

  SegArgs ga;
  ga.budgets = sa.budgets; ga.evict_mx = ma.evict_mx; ga.evict_nn = ma.evict_nn;
  ga.seg_start = (int32_t*)(X + c->slay.seg_start); ga.seg_items = (int32_t*)(X + c->slay.seg_items);
  ga.seg_tmp = (int32_t*)(X + c->slay.seg_tmp);
  ga.tau = sa.tau; ga.counters = sa.counters; ga.status = sa.status;
  ga.plen = sa.plen;
  ga.L = L; ga.layer = layer; ga.B = B; ga.Hkv = Hkv; ga.P = P; ga.seg_stride = seg_stride;
  ga.tau_override = g.tau_override;
  // counts / cursors per retained slot, later the radix histograms (32 warps x 64 digits)
  const size_t seg_sm = (size_t)max(maxS + 1, 32 * 64) * sizeof(int);
  e = cudaFuncSetAttribute(segment_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)(seg_sm > 48 * 1024 ? seg_sm : 48 * 1024));
  if (e != cudaSuccess) return e;
  segment_kernel<<<n_slices, 1024, seg_sm, st>>>(ga);

  MergeArgs mg;
  mg.budgets = sa.budgets; mg.row_off = sa.row_off; mg.evict_idx = sa.evict_idx; mg.evict_mx = ma.evict_mx;
  mg.seg_start = ga.seg_start; mg.seg_items = ga.seg_items; mg.rnorm = sa.rnorm;
  mg.plen = sa.plen;
  mg.L = L; mg.layer = layer; mg.Hkv = Hkv; mg.P = P; mg.seg_stride = seg_stride; mg.average = g.merge_policy;
  mg.value_feature = g.sim_feature; mg.status = sa.status;
  constexpr int LPR = D / Elem<T>::kPerVec;
  const int rows_per_cta = 256 / LPR;
  dim3 mgrid((maxS + rows_per_cta - 1) / rows_per_cta, n_slices);
  merge_kernel<T, D><<<mgrid, 256, 0, st>>>(mg, (const T*)K, (const T*)V, kpool, vpool);
  return cudaGetLastError();
}

cudaError_t launch_prefill_compress(const d2o_ctx* c, int layer, const void* K, const void* V, cudaStream_t st, int lane) {
  const int d = c->cfg.d_head;
  switch (c->cfg.dtype) {
    case D2O_F32: return d == 64 ? run_prefill<float, 64>(c, layer, K, V, st, lane) : run_prefill<float, 128>(c, layer, K, V, st, lane);
    case D2O_F16: return d == 64 ? run_prefill<__half, 64>(c, layer, K, V, st, lane) : run_prefill<__half, 128>(c, layer, K, V, st, lane);
    default: return d == 64 ? run_prefill<__nv_bfloat16, 64>(c, layer, K, V, st, lane)
                            : run_prefill<__nv_bfloat16, 128>(c, layer, K, V, st, lane);
  }
}

}  // namespace d2o
