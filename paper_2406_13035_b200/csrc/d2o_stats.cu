// Layer-level operation (Section 4.1): column sums of the causal prompt attention (Eq. 4 / Eq. 6
// case 1), the density F_v = Var(s) per query head, and the inverse-variance-softmax budgets
// (Eq. 5, Appendix A.2).
//
// Kernels in this file
//   lse_kernel      row normalisers log sum_j exp(q_i.k_j/sqrt(d)) of the causal attention
//   colsum_kernel   s_j = sum_{i>=j} exp(q_i.k_j/sqrt(d) - lse_i); one CTA owns a block of
//                   columns and walks down the rows, so the column reduction needs neither
//                   atomics nor scratch and is bit-reproducible
//   density_kernel  warp-shuffle mean / variance of s per query head (double accumulation)
//   budget_kernel   Eq. 5 with clamping and exact-sum integerisation, one thread per sequence
// The two attention sweeps here are the generic FFMA implementation (any dtype, fp32 math);
// 16-bit inputs take the tensor-core path of d2o_colsum_tc.cu.
#include <math.h>

#include "d2o_common.cuh"

namespace d2o {

constexpr int kTile = 64;        // rows and columns per CTA tile
constexpr int kStatThreads = 256;

// Loads a [64 x D] tile (rows row0.., zero beyond n_rows) transposed into smem as t[k][r], times `mul`.
template <typename T, int D>
__device__ __forceinline__ void load_tile_transposed(float* t, const T* base, int row0, int n_rows, float mul) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int VPR = D / EPV;                       // vectors per row
  const int r = threadIdx.x % kTile;
  for (int vi = threadIdx.x / kTile; vi < VPR; vi += kStatThreads / kTile) {
    float f[EPV];
    if (row0 + r < n_rows) {
      uint4 v = ld_global_v4(base + (size_t)(row0 + r) * D + vi * EPV);
      Elem<T>::unpack(v, f);
    } else {
#pragma unroll
      for (int i = 0; i < EPV; ++i) f[i] = 0.f;
    }
#pragma unroll
    for (int i = 0; i < EPV; ++i) t[(vi * EPV + i) * kTile + r] = f[i] * mul;
  }
}

// 4x4 register tile of S = Q K^T for this thread: rows ty*4.., cols tx*4..
template <int D>
__device__ __forceinline__ void tile_dot(const float* qt, const float* kt, int ty, int tx, float s[4][4]) {
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) s[r][c] = 0.f;
#pragma unroll 8
  for (int k = 0; k < D; ++k) {
    const float4 a = *reinterpret_cast<const float4*>(qt + k * kTile + ty * 4);
    const float4 b = *reinterpret_cast<const float4*>(kt + k * kTile + tx * 4);
    const float av[4] = {a.x, a.y, a.z, a.w};
    const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) s[r][c] = fmaf(av[r], bv[c], s[r][c]);
  }
}

// lse2[b,hq,i] = log2 sum_{j<=i} 2^{(q_i.k_j) * scale * log2e}, stored as natural log.
template <typename T, int D>
__global__ void __launch_bounds__(kStatThreads)
lse_kernel(const T* __restrict__ Q, const T* __restrict__ K, float* __restrict__ lse, int Pmax, int Hq, int group,
           const int32_t* __restrict__ plen) {
  extern __shared__ __align__(16) float smem[];
  float* qt = smem;
  float* kt = smem + D * kTile;
  const int it = gridDim.x - 1 - blockIdx.x;          // heaviest row tiles first
  const int bh = blockIdx.y;
  const int b = bh / Hq, hq = bh % Hq;
  const int P = plen ? plen[b] : Pmax;                 // this sequence's prompt length; tensors are laid out for Pmax
  if (it * kTile >= P) return;
  const int Hkv = Hq / group;
  const T* q = Q + ((size_t)b * Hq + hq) * (size_t)Pmax * D;
  const T* k = K + ((size_t)b * Hkv + hq / group) * (size_t)Pmax * D;
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
  const float mul = (D == 64 ? 0.125f : 0.08838834764831845f) * kLog2e;
  load_tile_transposed<T, D>(qt, q, it * kTile, P, mul);
  float m[4], l[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) { m[r] = -INFINITY; l[r] = 0.f; }
  for (int jt = 0; jt <= it; ++jt) {
    __syncthreads();
    load_tile_transposed<T, D>(kt, k, jt * kTile, P, 1.0f);
    __syncthreads();
    float s[4][4];
    tile_dot<D>(qt, kt, ty, tx, s);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = it * kTile + ty * 4 + r;
      float mx = m[r];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int col = jt * kTile + tx * 4 + c;
        if (col > row) s[r][c] = -INFINITY;
        mx = fmaxf(mx, s[r][c]);
      }
      if (mx > -INFINITY) {
        float add = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) add += exp2f(s[r][c] - mx);
        l[r] = l[r] * exp2f(m[r] - mx) + add;
        m[r] = mx;
      }
    }
  }
  // combine the 16 threads (tx) that share a row: contiguous lanes
#pragma unroll
  for (int r = 0; r < 4; ++r) {
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
      const float mo = __shfl_xor_sync(0xffffffffu, m[r], o);
      const float lo = __shfl_xor_sync(0xffffffffu, l[r], o);
      const float mn = fmaxf(m[r], mo);
      const float a = (m[r] > -INFINITY) ? l[r] * exp2f(m[r] - mn) : 0.f;
      const float bb = (mo > -INFINITY) ? lo * exp2f(mo - mn) : 0.f;
      l[r] = a + bb;
      m[r] = mn;
    }
    const int row = it * kTile + ty * 4 + r;
    if (tx == 0 && row < P) lse[((size_t)b * Hq + hq) * Pmax + row] = (m[r] + log2f(l[r])) * 0.6931471805599453f;
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kStatThreads)
colsum_kernel(const T* __restrict__ Q, const T* __restrict__ K, const float* __restrict__ lse,
              float* __restrict__ colsum, int Pmax, int Hq, int group, const int32_t* __restrict__ plen) {
  extern __shared__ __align__(16) float smem[];
  float* qt = smem;
  float* kt = smem + D * kTile;
  float* lse2 = kt + D * kTile;                        // [64]
  double* red = reinterpret_cast<double*>(lse2 + kTile);  // [16][64]
  const int jt = blockIdx.x;                          // column tile 0 has the most rows: first
  const int bh = blockIdx.y;
  const int b = bh / Hq, hq = bh % Hq;
  const int P = plen ? plen[b] : Pmax;
  const int nT = (P + kTile - 1) / kTile;
  if (jt >= nT) return;
  const int Hkv = Hq / group;
  const T* q = Q + ((size_t)b * Hq + hq) * (size_t)Pmax * D;
  const T* k = K + ((size_t)b * Hkv + hq / group) * (size_t)Pmax * D;
  const float* ls = lse + ((size_t)b * Hq + hq) * Pmax;
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
  const float mul = (D == 64 ? 0.125f : 0.08838834764831845f) * kLog2e;
  load_tile_transposed<T, D>(kt, k, jt * kTile, P, 1.0f);
  double acc[4] = {0.0, 0.0, 0.0, 0.0};
  for (int it = jt; it < nT; ++it) {
    __syncthreads();
    load_tile_transposed<T, D>(qt, q, it * kTile, P, mul);
    if (threadIdx.x < kTile) {
      const int row = it * kTile + threadIdx.x;
      lse2[threadIdx.x] = row < P ? ls[row] * kLog2e : INFINITY;    // +inf -> probability 0 for padding rows
    }
    __syncthreads();
    float s[4][4];
    tile_dot<D>(qt, kt, ty, tx, s);
    float p[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = it * kTile + ty * 4 + r;
      const float lr = lse2[ty * 4 + r];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int col = jt * kTile + tx * 4 + c;
        p[r][c] = (col <= row) ? exp2f(s[r][c] - lr) : 0.f;
      }
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[c] += (double)((p[0][c] + p[1][c]) + (p[2][c] + p[3][c]));
  }
  __syncthreads();
#pragma unroll
  for (int c = 0; c < 4; ++c) red[ty * kTile + tx * 4 + c] = acc[c];
  __syncthreads();
  if (threadIdx.x < kTile) {
    double t = 0.0;
#pragma unroll
    for (int y = 0; y < 16; ++y) t += red[y * kTile + threadIdx.x];
    const int col = jt * kTile + threadIdx.x;
    if (col < P) colsum[((size_t)b * Hq + hq) * Pmax + col] = (float)t;
  }
}

// F[b, layer, hq] = (1/P) sum_j (s_j - mean)^2, mean = (1/P) sum_j s_j   (Eq. 4; population variance)
__global__ void __launch_bounds__(256)
density_kernel(const float* __restrict__ colsum, double* __restrict__ density, int Pmax, int Hq, int L, int layer,
               const int32_t* __restrict__ plen) {
  __shared__ double part[8];
  __shared__ double mean_s;
  const int bh = blockIdx.x;
  const int b = bh / Hq, hq = bh % Hq;
  const int P = plen ? plen[b] : Pmax;
  const float* s = colsum + (size_t)bh * Pmax;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double t = 0.0;
  for (int j = threadIdx.x; j < P; j += blockDim.x) t += (double)s[j];
  t = warp_sum(t);
  if (lane == 0) part[warp] = t;
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0.0;
    for (int w = 0; w < 8; ++w) a += part[w];
    mean_s = a / (double)P;
  }
  __syncthreads();
  const double mean = mean_s;
  t = 0.0;
  for (int j = threadIdx.x; j < P; j += blockDim.x) { const double dlt = (double)s[j] - mean; t += dlt * dlt; }
  t = warp_sum(t);
  __syncthreads();
  if (lane == 0) part[warp] = t;
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0.0;
    for (int w = 0; w < 8; ++w) a += part[w];
    density[((size_t)b * L + layer) * Hq + hq] = a / (double)P;
  }
}

// Cache sizes from the densities.  budget_rule 0 (Eq. 5): S_l = clip(lambda * w_l, S_min, S_max) with
// sum_l S_l = S_tot, then floor + largest remainder; rule 1 (per-head sizes of Appendix A.5): the same over the
// (layer, KV head) units; rule 2 (exponential-decay allocation of the ablation): S_l = round(mean_h exp(-F/gamma) P),
// clamped, no fixed total.  One thread per sequence; its work arrays (w, kinks, x) live in dynamic shared memory.
// Output tables are [B, L, Hkv]; the per-layer rules give every KV head of a layer the same size.
__device__ inline double clipd(double v, double lo, double hi) { return v < lo ? lo : (v > hi ? hi : v); }

__global__ void budget_kernel(const double* __restrict__ density, int B, int L, int H, int Hkv, int Pmax, double rho,
                              int min_budget, int max_budget_cfg, double gamma, int head_reduce, int budget_rule,
                              int n_sink, int window, double nm_ratio, int32_t* __restrict__ budgets,
                              int32_t* __restrict__ windows, int64_t* __restrict__ row_off, uint32_t* status_word,
                              const int32_t* __restrict__ plen) {
  extern __shared__ __align__(16) double dsm[];
  const int n = budget_rule == 1 ? L * Hkv : L;                       // allocation units
  const int G = H / Hkv;
  double* w = dsm + (size_t)threadIdx.x * 4 * n;
  double* kinks = w + n;        // [2n]
  double* x = kinks + 2 * n;    // [n]
  const double lo = (double)min_budget;
  for (int b = threadIdx.x; b < B; b += blockDim.x) {
    const int P = plen ? plen[b] : Pmax;                              // this sequence's prompt length
    const int max_budget = max_budget_cfg > 0 ? max_budget_cfg : P;   // no clamp given: a layer cannot hold more than the prompt
    const double hi = (double)max_budget;
    const long long S_tot = (long long)floor(rho * (double)n * (double)P + 0.5);
    const double* F = density + (size_t)b * L * H;
    int32_t* bud = budgets + (size_t)b * L * Hkv;
    // unit u -> its (first) entry of the [L, Hkv] table
    auto slot_of = [&](int u) { return budget_rule == 1 ? u : u * Hkv; };
    if (budget_rule == 2) {
      for (int l = 0; l < L; ++l) {
        double a = 0.0;
        for (int h = 0; h < H; ++h) a = __dadd_rn(a, exp(-__ddiv_rn(F[l * H + h], gamma)));
        const double s = floor(__dadd_rn(__dmul_rn(__ddiv_rn(a, (double)H), (double)P), 0.5));
        bud[l * Hkv] = (int32_t)clipd(s, lo, hi);
      }
    } else {
      if (budget_rule == 1) {
        double fmin = F[0];
        for (int i = 1; i < L * H; ++i) fmin = fmin < F[i] ? fmin : F[i];
        for (int u = 0; u < n; ++u) {
          double a = 0.0;
          for (int g = 0; g < G; ++g) a = __dadd_rn(a, exp(-__ddiv_rn(__dadd_rn(F[u * G + g], -fmin), gamma)));
          w[u] = a;
        }
      } else if (head_reduce == 0) {
        double fmin = F[0];
        for (int i = 1; i < L * H; ++i) fmin = fmin < F[i] ? fmin : F[i];
        for (int l = 0; l < L; ++l) {
          double a = 0.0;
          for (int h = 0; h < H; ++h) a = __dadd_rn(a, exp(-__ddiv_rn(__dadd_rn(F[l * H + h], -fmin), gamma)));
          w[l] = a;
        }
      } else if (head_reduce == 2) {
        // reciprocal of the variance, per head (a zero variance counts as the smallest positive one)
        for (int l = 0; l < L; ++l) {
          double a = 0.0;
          for (int h = 0; h < H; ++h) {
            const double f = F[l * H + h];
            a = __dadd_rn(a, __ddiv_rn(1.0, f > 1e-300 ? f : 1e-300));
          }
          w[l] = a;
        }
      } else {
        double fmin = INFINITY;
        for (int l = 0; l < L; ++l) {
          double a = 0.0;
          for (int h = 0; h < H; ++h) a = __dadd_rn(a, F[l * H + h]);
          x[l] = __ddiv_rn(a, (double)H);
          fmin = fmin < x[l] ? fmin : x[l];
        }
        if (head_reduce == 1) {
          for (int l = 0; l < L; ++l) w[l] = exp(-__ddiv_rn(__dadd_rn(x[l], -fmin), gamma));
        } else {
          for (int l = 0; l < L; ++l) w[l] = __ddiv_rn(1.0, x[l] > 1e-300 ? x[l] : 1e-300);
        }
      }
      for (int u = 0; u < n; ++u) w[u] = w[u] > 1e-300 ? (w[u] < 1e300 ? w[u] : 1e300) : 1e-300;
      // kinks of the piecewise-linear total(lambda), ascending (insertion sort)
      int nk = 0;
      for (int u = 0; u < n; ++u) {
        const double cand[2] = {__ddiv_rn(lo, w[u]), __ddiv_rn(hi, w[u])};
        for (int c = 0; c < 2; ++c) {
          int i = nk++;
          while (i > 0 && kinks[i - 1] > cand[c]) { kinks[i] = kinks[i - 1]; --i; }
          kinks[i] = cand[c];
        }
      }
      auto total = [&](double lam) {
        double t = 0.0;
        for (int u = 0; u < n; ++u) t = __dadd_rn(t, clipd(__dmul_rn(lam, w[u]), lo, hi));
        return t;
      };
      // total() is non-decreasing: the first kink that reaches S_tot, by bisection
      int k = 0, k_hi = nk;
      while (k < k_hi) {
        const int mid = (k + k_hi) >> 1;
        if (total(kinks[mid]) < (double)S_tot) k = mid + 1; else k_hi = mid;
      }
      double lam;
      if (k == 0) lam = kinks[0];
      else if (k == nk) lam = kinks[nk - 1];
      else {
        const double a = kinks[k - 1], bb = kinks[k];
        const double mid = __dmul_rn(0.5, __dadd_rn(a, bb));
        double fixed = 0.0, wf = 0.0;
        for (int u = 0; u < n; ++u) {
          const double v = __dmul_rn(mid, w[u]);
          if (v > lo && v < hi) wf = __dadd_rn(wf, w[u]);
          else fixed = __dadd_rn(fixed, clipd(v, lo, hi));
        }
        lam = wf > 0.0 ? __ddiv_rn(__dadd_rn((double)S_tot, -fixed), wf) : bb;
        lam = lam < a ? a : (lam > bb ? bb : lam);
      }
      long long sum = 0;
      for (int u = 0; u < n; ++u) {
        x[u] = clipd(__dmul_rn(lam, w[u]), lo, hi);
        const double fl = floor(x[u]);
        bud[slot_of(u)] = (int32_t)fl;
        x[u] = x[u] - fl;                                   // remainder
        sum += (long long)fl;
      }
      long long left = S_tot - sum;
      if (left < 0 || left > n) { report_error(status_word, D2O_ERR_STATE, 0xB0000000u | (uint32_t)b); left = 0; }
      while (left > 0) {                                     // largest remainder first, ties -> lower unit
        int best = -1;
        for (int u = 0; u < n; ++u)
          if (x[u] >= 0.0 && bud[slot_of(u)] < max_budget && (best < 0 || x[u] > x[best])) best = u;
        if (best < 0) { report_error(status_word, D2O_ERR_STATE, 0xB1000000u | (uint32_t)b); break; }
        bud[slot_of(best)] += 1;
        x[best] = -1.0;                                      // taken
        --left;
      }
    }
    if (budget_rule != 1) {                                  // one size per layer: every KV head gets it
      for (int l = 0; l < L; ++l)
        for (int h = 1; h < Hkv; ++h) bud[l * Hkv + h] = bud[l * Hkv];
    }
    if (windows) {
      for (int i = 0; i < L * Hkv; ++i) {
        const int S = bud[i];
        const int T = n_sink < S ? n_sink : S;
        int M = window > 0 ? window : (int)floor((double)(S - T) / (1.0 + nm_ratio) + 0.5);
        M = M < 0 ? 0 : (M > S - T ? S - T : M);
        windows[(size_t)b * L * Hkv + i] = M;
      }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0 && row_off) {                       // cache rows laid out layer-major, then sequence, then head
    long long o = 0;
    for (int l = 0; l < L; ++l)
      for (int b = 0; b < B; ++b)
        for (int h = 0; h < Hkv; ++h) {
          const size_t i = ((size_t)b * L + l) * Hkv + h;
          row_off[i] = o;
          o += (long long)slice_stride(budgets[i]);
        }
  }
}

template <typename T, int D>
static cudaError_t run_stats(const d2o_ctx* c, int layer, const void* Q, const void* K, const float* lse_in,
                             cudaStream_t st, int lane) {
  const d2o_config& g = c->cfg;
  const int P = g.prompt_len, Hq = g.n_q_heads, B = g.batch;
  const int nT = (P + kTile - 1) / kTile;
  float* colsum = (float*)(c->state + c->lay.colsum) + (size_t)layer * B * Hq * P;
  double* density = (double*)(c->state + c->lay.density);
  const int32_t* plen = (const int32_t*)(c->state + c->lay.plen);
  if (c->stats_path == 0 && colsum_tc_supported(&g)) {
    cudaError_t e = launch_colsum_tc(c, Q, K, lse_in, colsum, st, lane);
    if (e != cudaSuccess) return e;
    density_kernel<<<B * Hq, 256, 0, st>>>(colsum, density, P, Hq, g.n_layers, layer, plen);
    return cudaGetLastError();
  }
  const float* lse = lse_in;
  dim3 grid(nT, B * Hq);
  if (!lse) {
    float* lse_buf = (float*)(c->scratch + c->slay.lse + (size_t)lane * c->slay.lse_stride);
    const size_t sm = (size_t)2 * D * kTile * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(lse_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    lse_kernel<T, D><<<grid, kStatThreads, sm, st>>>((const T*)Q, (const T*)K, lse_buf, P, Hq, c->group, plen);
    lse = lse_buf;
  }
  const size_t sm2 = (size_t)2 * D * kTile * sizeof(float) + kTile * sizeof(float) + 16 * kTile * sizeof(double);
  cudaError_t e = cudaFuncSetAttribute(colsum_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm2);
  if (e != cudaSuccess) return e;
  colsum_kernel<T, D><<<grid, kStatThreads, sm2, st>>>((const T*)Q, (const T*)K, lse, colsum, P, Hq, c->group, plen);
  density_kernel<<<B * Hq, 256, 0, st>>>(colsum, density, P, Hq, g.n_layers, layer, plen);
  return cudaGetLastError();
}

cudaError_t launch_layer_stats(const d2o_ctx* c, int layer, const void* Q, const void* K, const float* lse,
                               cudaStream_t st, int lane) {
  const int d = c->cfg.d_head;
  switch (c->cfg.dtype) {
    case D2O_F32: return d == 64 ? run_stats<float, 64>(c, layer, Q, K, lse, st, lane) : run_stats<float, 128>(c, layer, Q, K, lse, st, lane);
    case D2O_F16: return d == 64 ? run_stats<__half, 64>(c, layer, Q, K, lse, st, lane) : run_stats<__half, 128>(c, layer, Q, K, lse, st, lane);
    default: return d == 64 ? run_stats<__nv_bfloat16, 64>(c, layer, Q, K, lse, st, lane)
                            : run_stats<__nv_bfloat16, 128>(c, layer, Q, K, lse, st, lane);
  }
}

cudaError_t launch_budgets(const double* density, int B, int L, int H, int Hkv, int P, float rho, int min_budget,
                           int max_budget, float gamma, int head_reduce, int budget_rule, int n_sink, int window,
                           float nm_ratio, int32_t* budgets, int32_t* windows, int64_t* row_off, uint32_t* status_word,
                           const int32_t* plen, cudaStream_t st) {
  const size_t n_units = budget_rule == 1 ? (size_t)L * Hkv : (size_t)L;
  const size_t per_thread = 4 * n_units * sizeof(double);
  int threads = B < 32 ? B : 32;
  while (threads > 1 && per_thread * threads > 160 * 1024) threads /= 2;
  const size_t sm = per_thread * threads;
  if (sm > 200 * 1024) return cudaErrorInvalidValue;          // more allocation units than the work arrays hold
  cudaError_t e = cudaFuncSetAttribute(budget_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
  if (e != cudaSuccess) return e;
  budget_kernel<<<1, threads, sm, st>>>(density, B, L, H, Hkv, P, (double)rho, min_budget, max_budget, (double)gamma,
                                        head_reduce, budget_rule, n_sink, window, (double)nm_ratio, budgets, windows,
                                        row_off, status_word, plen);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------ allocation-free variant
// Scratch for the row normalisers of d2o_layer_stats_static: part of the library image, one copy per GPU.
static __device__ __align__(256) float g_static_lse[D2O_STATIC_LSE_FLOATS];
constexpr int kMaxDevices = 64;
static float* g_static_lse_addr[kMaxDevices];        // device address of g_static_lse, per device (host-side cache)

template <typename T, int D>
static cudaError_t run_stats_static(const void* Q, const void* K, float* lse_buf, float* colsum, double* density, int B,
                                    int Hq, int group, int P, cudaStream_t st) {
  const int nT = (P + kTile - 1) / kTile;
  dim3 grid(nT, B * Hq);
  const size_t sm = (size_t)2 * D * kTile * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(lse_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
  if (e != cudaSuccess) return e;
  lse_kernel<T, D><<<grid, kStatThreads, sm, st>>>((const T*)Q, (const T*)K, lse_buf, P, Hq, group, nullptr);
  const size_t sm2 = sm + kTile * sizeof(float) + 16 * kTile * sizeof(double);
  e = cudaFuncSetAttribute(colsum_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm2);
  if (e != cudaSuccess) return e;
  colsum_kernel<T, D><<<grid, kStatThreads, sm2, st>>>((const T*)Q, (const T*)K, lse_buf, colsum, P, Hq, group, nullptr);
  density_kernel<<<B * Hq, 256, 0, st>>>(colsum, density, P, Hq, 1, 0, nullptr);
  return cudaGetLastError();
}

}  // namespace d2o

extern "C" d2o_status d2o_layer_stats_static(int32_t dtype, int32_t d_head, int32_t batch, int32_t n_q_heads,
                                             int32_t n_kv_heads, int32_t prompt_len, const void* Q, const void* K,
                                             float* colsum, double* density, void* stream) {
  using namespace d2o;
  if (dtype != D2O_F32 && dtype != D2O_F16 && dtype != D2O_BF16) return D2O_ERR_UNSUPPORTED;
  if (d_head != 64 && d_head != 128) return D2O_ERR_UNSUPPORTED;
  if (batch < 1 || n_q_heads < 1 || n_kv_heads < 1 || prompt_len < 1 || n_q_heads % n_kv_heads != 0)
    return D2O_ERR_INVALID_ARG;
  auto aligned16 = [](const void* p) { return p && (((uintptr_t)p & 15) == 0); };
  if (!aligned16(Q) || !aligned16(K) || !aligned16(colsum) || !density || ((uintptr_t)density & 7)) return D2O_ERR_INVALID_ARG;
  if ((unsigned long long)batch * n_q_heads * prompt_len > (unsigned long long)D2O_STATIC_LSE_FLOATS)
    return D2O_ERR_TOO_LARGE;
  if ((long long)batch * n_q_heads > 65535) return D2O_ERR_TOO_LARGE;      // one grid row per (sequence, head)
  // set-up, once per device: in host code `g_static_lse` is only a handle, the kernels need its device address
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return record_cuda_error(e, "cudaGetDevice");
  if (dev < 0 || dev >= kMaxDevices) return D2O_ERR_UNSUPPORTED;
  float* lse_buf = __atomic_load_n(&g_static_lse_addr[dev], __ATOMIC_ACQUIRE);
  if (!lse_buf) {
    e = cudaGetSymbolAddress((void**)&lse_buf, g_static_lse);
    if (e != cudaSuccess || !lse_buf) return record_cuda_error(e, "cudaGetSymbolAddress(g_static_lse)");
    __atomic_store_n(&g_static_lse_addr[dev], lse_buf, __ATOMIC_RELEASE);     // every thread would store the same value
  }
  const int group = n_q_heads / n_kv_heads;
  cudaStream_t st = (cudaStream_t)stream;
  switch (dtype) {
    case D2O_F32:
      e = d_head == 64 ? run_stats_static<float, 64>(Q, K, lse_buf, colsum, density, batch, n_q_heads, group, prompt_len, st)
                       : run_stats_static<float, 128>(Q, K, lse_buf, colsum, density, batch, n_q_heads, group, prompt_len, st);
      break;
    case D2O_F16:
      e = d_head == 64 ? run_stats_static<__half, 64>(Q, K, lse_buf, colsum, density, batch, n_q_heads, group, prompt_len, st)
                       : run_stats_static<__half, 128>(Q, K, lse_buf, colsum, density, batch, n_q_heads, group, prompt_len, st);
      break;
    default:
      e = d_head == 64 ? run_stats_static<__nv_bfloat16, 64>(Q, K, lse_buf, colsum, density, batch, n_q_heads, group, prompt_len, st)
                       : run_stats_static<__nv_bfloat16, 128>(Q, K, lse_buf, colsum, density, batch, n_q_heads, group, prompt_len, st);
  }
  if (e != cudaSuccess) return record_cuda_error(e, "d2o_layer_stats_static launch");
  return D2O_OK;
}
