// Token generation (Section 3, Eq. 2-3; Section 4.2, Eq. 6-12): one fused kernel per decode step.
//
// One thread-block cluster handles one slice = (layer, sequence, KV head) with its G query heads.
// The slice's cache rows are split evenly over the CTAs of the cluster.  Each CTA
//   1. streams its K rows once from HBM (128-bit loads), keeps them in shared memory, and
//      computes the G logit vectors; the new token's key is row `len`;
//   2. publishes its softmax (max, sum), then streams its V rows once and accumulates
//      un-normalised outputs while the cluster barrier completes in the background;
//   3. turns its probabilities into accumulated scores (Eq. 6 case 2) and publishes its lowest
//      score outside the T sinks and the M most recent positions (Eq. 7-8: the victim candidate);
//      rank 0 combines the partial outputs;
//   4. reads the victim's key from its owner's shared memory (distributed shared memory) and takes
//      the cosine similarity with its own resident rows (Eq. 9); publishes its best neighbour;
//   5. tau_t = beta*max(U) + (1-beta)*tau_{t-1} (Eq. 10); at or above it the owner of the nearest
//      neighbour merges the victim into it with weights e^u/(e^u+e), e/(e^u+e) (Eq. 11-12);
//   6. the new token takes the victim's row.
// HBM traffic per step is one pass over K_c and V_c plus a few rows.  Cluster barriers are split
// into arrive / wait so that their latency overlaps the work that does not depend on the peers.
// The same kernel with COMPRESS=false is the uncompressed decode attention (steps 1-3 and an
// append), used as the comparison kernel.
#include <cooperative_groups.h>
#include <math.h>

#include "d2o_common.cuh"

namespace cg = cooperative_groups;

namespace d2o {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kMaxCluster = 8;

struct DecodeArgs {
  const int32_t* budgets; const int32_t* windows; const int64_t* row_off;   // [B, L]
  int32_t* pos; float* score; float* rnorm;                                  // pool-wide
  int32_t* len; float* tau;                                                  // [L, B, Hkv]
  unsigned long long* counters; uint32_t* status;
  int L, l0, B, Hkv, T, t;          // t = position of the token generated in this step
  float beta, tau_override;
  int chunk_cap;                    // rows per CTA the shared-memory arrays are sized for
  int res_rows;                     // K rows per CTA kept resident in shared memory
  // uncompressed mode
  int full_capacity, full_len;
};

template <int G, int D>
struct alignas(16) Exchange {        // the part of shared memory that peer CTAs read
  float m[G];
  float l[G];
  float acc[G][D];
  unsigned long long cand_min;       // victim candidate of this CTA: (score bits, 0x7fffffff - pos)
  unsigned long long cand_max;       // neighbour candidate: (ordered similarity bits, 0x7fffffff - pos)
  int cand_min_li, cand_max_li;      // their local row indices
  int pad[2];
};

__device__ __forceinline__ void cluster_arrive() { __syncwarp(); asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { __syncwarp(); asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// Block-wide extremum of a 64-bit key with the local row index of the winner (keys are unique per row).
template <bool MIN>
__device__ __forceinline__ void block_arg_extreme(unsigned long long key, int li, unsigned long long* s_key,
                                                   int* s_li, unsigned long long* out_key, int* out_li) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned long long w = MIN ? warp_min_u64(key) : warp_max_u64(key);
  const unsigned vote = __ballot_sync(0xffffffffu, key == w);
  const int src = __ffs(vote) - 1;
  const int wli = __shfl_sync(0xffffffffu, li, src);
  if (lane == 0) { s_key[warp] = w; s_li[warp] = wli; }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long b = s_key[0]; int bl = s_li[0];
    for (int i = 1; i < kDecWarps; ++i) {
      const bool better = MIN ? (s_key[i] < b) : (s_key[i] > b);
      if (better) { b = s_key[i]; bl = s_li[i]; }
    }
    *out_key = b; *out_li = bl;
  }
}

template <typename T, int D, int G, bool COMPRESS>
__global__ void __launch_bounds__(kDecThreads, (G <= 2 ? 3 : 2))
decode_kernel(DecodeArgs a, const T* __restrict__ q_in, const T* __restrict__ k_in, const T* __restrict__ v_in,
              T* __restrict__ out, T* __restrict__ kpool, T* __restrict__ vpool) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int LPR = D / EPV;                  // lanes that share one row (16-byte segment each)
  constexpr int NGRP = kDecThreads / LPR;       // rows in flight per CTA iteration
  using Xch = Exchange<G, D>;

  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int sl = blockIdx.x / C;                // slice index within the launch
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int grp = tid / LPR, lig = tid % LPR;
  const unsigned gmask = group_mask<LPR>();

  // ---- slice parameters
  int S, M, n_old, sidx = 0;
  int64_t row0;
  if (COMPRESS) {
    const int per_layer = a.B * a.Hkv;
    const int layer = a.l0 + sl / per_layer;
    const int bh = sl % per_layer;
    const int b = bh / a.Hkv, h = bh % a.Hkv;
    S = a.budgets[b * a.L + layer];
    M = a.windows[b * a.L + layer];
    row0 = a.row_off[b * a.L + layer] + (int64_t)h * S;
    sidx = (layer * a.B + b) * a.Hkv + h;
    n_old = a.len[sidx];
  } else {
    S = a.full_capacity; M = 0;
    row0 = (int64_t)sl * a.full_capacity;
    n_old = a.full_len;
  }
  const int n = n_old + 1;                                         // rows attended: cache + the new token
  const int chunk = (((n + C - 1) / C) + 7) & ~7;
  const int r0 = rank * chunk;
  const int cnt = max(0, min(n, r0 + chunk) - r0);                 // rows of this CTA
  const float tau_old = COMPRESS ? a.tau[sidx] : 0.f;
  const int Tn = a.T < S ? a.T : S;

  // ---- shared memory carve-up (identical in every CTA of the cluster, so peers can address it)
  extern __shared__ __align__(16) unsigned char dsm[];
  Xch* xch = reinterpret_cast<Xch*>(dsm);
  float* red = reinterpret_cast<float*>(dsm + sizeof(Xch));        // [warps][G][D]
  float* pl = red + kDecWarps * G * D;                              // [G][chunk_cap] logits -> probabilities
  float* sc = pl + (size_t)G * a.chunk_cap;                         // [chunk_cap] scores
  float* rn = sc + a.chunk_cap;                                     // [chunk_cap] inverse key norms
  int* ps = reinterpret_cast<int*>(rn + a.chunk_cap);               // [chunk_cap] positions
  uint4* newkv = reinterpret_cast<uint4*>(ps + a.chunk_cap);        // [2][LPR] staging of the new token's row
  uint4* ks = newkv + 2 * LPR;                                      // [res_rows][LPR]
  __shared__ float s_red[kDecWarps][G];
  __shared__ unsigned long long s_key[kDecWarps];
  __shared__ int s_li[kDecWarps];
  __shared__ float s_fac[G];

  const T* k_new = k_in + (size_t)sl * D;
  const T* v_new = v_in + (size_t)sl * D;
  auto k_src = [&](int li) -> const T* {       // global source of local row li
    const int gi = r0 + li;
    return gi < n_old ? kpool + (row0 + gi) * D : k_new;
  };
  auto v_src = [&](int li) -> const T* {
    const int gi = r0 + li;
    return gi < n_old ? vpool + (row0 + gi) * D : v_new;
  };

  // ---- query fragments, pre-scaled by log2(e)/sqrt(d)
  float qf[G][EPV];
  {
    const float mul = (D == 64 ? 0.125f : 0.08838834764831845f) * kLog2e;
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float f[EPV];
      Elem<T>::unpack(ld_global_v4(q_in + ((size_t)sl * G + g) * D + lig * EPV), f);
#pragma unroll
      for (int e = 0; e < EPV; ++e) qf[g][e] = f[e] * mul;
    }
  }
  // ---- per-row metadata
  if (COMPRESS) {
    for (int li = tid; li < cnt; li += kDecThreads) {
      const int gi = r0 + li;
      ps[li] = gi < n_old ? a.pos[row0 + gi] : a.t;
      sc[li] = gi < n_old ? a.score[row0 + gi] : 0.f;
      if (gi < n_old) rn[li] = a.rnorm[row0 + gi];                  // the new row's norm is computed in the K pass
    }
  }
  // ---- 1. K pass: logits, keep rows in shared memory
  constexpr int U = 4;
  for (int li0 = grp; li0 < cnt; li0 += NGRP * U) {
    uint4 kv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int li = li0 + u * NGRP;
      if (li < cnt) kv[u] = ld_stream_v4(k_src(li) + lig * EPV);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int li = li0 + u * NGRP;
      if (li < cnt) {
        if (COMPRESS && li < a.res_rows) ks[(size_t)li * LPR + lig] = kv[u];
        float f[EPV];
        Elem<T>::unpack(kv[u], f);
        float dot[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float s = 0.f;
#pragma unroll
          for (int e = 0; e < EPV; ++e) s = fmaf(qf[g][e], f[e], s);
          dot[g] = s;
        }
#pragma unroll
        for (int g = 0; g < G; ++g) dot[g] = group_sum<LPR>(dot[g], gmask);
        if (lig == 0) {
#pragma unroll
          for (int g = 0; g < G; ++g) pl[(size_t)g * a.chunk_cap + li] = dot[g];
        }
        if (COMPRESS && r0 + li == n_old) {                         // the new token: its norm and a staging copy
          float ss = 0.f;
#pragma unroll
          for (int e = 0; e < EPV; ++e) ss = fmaf(f[e], f[e], ss);
          ss = group_sum<LPR>(ss, gmask);
          if (lig == 0) rn[li] = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
          newkv[lig] = kv[u];
        }
      }
    }
  }
  __syncthreads();
  // ---- local softmax statistics per query head
  float m_loc[G], l_loc[G];
  {
    float mx[G];
#pragma unroll
    for (int g = 0; g < G; ++g) mx[g] = -INFINITY;
    for (int li = tid; li < cnt; li += kDecThreads) {
#pragma unroll
      for (int g = 0; g < G; ++g) mx[g] = fmaxf(mx[g], pl[(size_t)g * a.chunk_cap + li]);
    }
#pragma unroll
    for (int g = 0; g < G; ++g) { mx[g] = warp_max(mx[g]); if (lane == 0) s_red[warp][g] = mx[g]; }
    __syncthreads();
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float t = s_red[0][g];
#pragma unroll
      for (int w = 1; w < kDecWarps; ++w) t = fmaxf(t, s_red[w][g]);
      m_loc[g] = t;
    }
    __syncthreads();
    float sum[G];
#pragma unroll
    for (int g = 0; g < G; ++g) sum[g] = 0.f;
    for (int li = tid; li < cnt; li += kDecThreads) {
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float p = exp2f(pl[(size_t)g * a.chunk_cap + li] - m_loc[g]);
        pl[(size_t)g * a.chunk_cap + li] = p;
        sum[g] += p;
      }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) { sum[g] = warp_sum(sum[g]); if (lane == 0) s_red[warp][g] = sum[g]; }
    __syncthreads();
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < kDecWarps; ++w) t += s_red[w][g];
      l_loc[g] = t;
    }
#pragma unroll
    for (int g = 0; g < G; ++g)
      if (tid == g) { xch->m[g] = m_loc[g]; xch->l[g] = l_loc[g]; }
  }
  cluster_arrive();                                                  // #1 (max, sum) published; completes during the V pass
  // ---- 2. V pass: un-normalised outputs
  {
    float acc[G][EPV];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
      for (int e = 0; e < EPV; ++e) acc[g][e] = 0.f;
    for (int li0 = grp; li0 < cnt; li0 += NGRP * U) {
      uint4 vv[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int li = li0 + u * NGRP;
        if (li < cnt) vv[u] = ld_stream_v4(v_src(li) + lig * EPV);
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int li = li0 + u * NGRP;
        if (li < cnt) {
          float f[EPV];
          Elem<T>::unpack(vv[u], f);
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const float p = pl[(size_t)g * a.chunk_cap + li];
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc[g][e] = fmaf(p, f[e], acc[g][e]);
          }
          if (COMPRESS && r0 + li == n_old) newkv[LPR + lig] = vv[u];
        }
      }
    }
    // combine the row groups of a warp, then the warps
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
      for (int g = 0; g < G; ++g)
#pragma unroll
        for (int e = 0; e < EPV; ++e) acc[g][e] += __shfl_xor_sync(0xffffffffu, acc[g][e], o);
    }
    if (lane < LPR) {
#pragma unroll
      for (int g = 0; g < G; ++g)
#pragma unroll
        for (int e = 0; e < EPV; ++e) red[((size_t)warp * G + g) * D + lane * EPV + e] = acc[g][e];
    }
    __syncthreads();
    for (int i = tid; i < G * D; i += kDecThreads) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < kDecWarps; ++w) t += red[(size_t)w * G * D + i];
      xch->acc[i / D][i % D] = t;
    }
  }
  cluster_wait();                                                    // #1
  // ---- 3. global softmax normaliser from the peers' (max, sum)
  float m_star[G], l_star[G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    float ms = -INFINITY;
    for (int r = 0; r < C; ++r) ms = fmaxf(ms, cluster.map_shared_rank(xch, r)->m[g]);
    float ls = 0.f;
    for (int r = 0; r < C; ++r) {
      const Xch* x = cluster.map_shared_rank(xch, r);
      ls += x->l[g] * exp2f(x->m[g] - ms);
    }
    m_star[g] = ms; l_star[g] = ls;
  }
  const bool evict = COMPRESS && (n > S);
  unsigned long long my_min = ~0ull; int my_min_li = -1;
  if (COMPRESS) {
    // accumulated attention (Eq. 6 case 2): add this step's probabilities, summed over the G heads;
    // victim candidate: lowest score outside sinks and window, ties -> latest position
    float fac[G];
#pragma unroll
    for (int g = 0; g < G; ++g) fac[g] = exp2f(m_loc[g] - m_star[g]) / l_star[g];
    for (int li = tid; li < cnt; li += kDecThreads) {
      float p = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g) p = fmaf(pl[(size_t)g * a.chunk_cap + li], fac[g], p);
      const float s_new = sc[li] + p;
      sc[li] = s_new;
      const int pz = ps[li];
      if (evict && pz >= Tn && pz <= a.t - M) {
        const unsigned long long key = ((unsigned long long)float_ord(s_new) << 32) | (uint32_t)(0x7fffffff - pz);
        if (key < my_min) { my_min = key; my_min_li = li; }
      }
    }
    if (evict) block_arg_extreme<true>(my_min, my_min_li, s_key, s_li, &xch->cand_min, &xch->cand_min_li);
  }
  cluster_arrive();                                                  // #2 partial outputs (and victim candidates) published
  const int new_rank = n_old / chunk;                                // CTA that holds the new token's row
  const int new_li = n_old - new_rank * chunk;
  if (COMPRESS) {
    // score write-back overlaps the barrier; the victim's row is overwritten by the new token at the very end
    for (int li = tid; li < cnt; li += kDecThreads) {
      const int gi = r0 + li;
      if (gi < n_old || !evict) a.score[row0 + gi] = sc[li];
    }
  }
  cluster_wait();                                                    // #2
  if (rank == 0) {
    for (int i = tid; i < G * D; i += kDecThreads) {
      const int g = i / D, dd = i % D;
      float num = 0.f;
      for (int r = 0; r < C; ++r) {
        const Xch* x = cluster.map_shared_rank(xch, r);
        num = fmaf(x->acc[g][dd], exp2f(x->m[g] - m_star[g]), num);
      }
      out[((size_t)sl * G + g) * D + dd] = Elem<T>::from_float(num / l_star[g]);
    }
  }
  if (!evict) {
    // append the new token's row (cache not full, or uncompressed mode)
    if (rank == new_rank && grp == 0) {
      if (COMPRESS) {
        *reinterpret_cast<uint4*>(kpool + (row0 + n_old) * D + lig * EPV) = newkv[lig];
        *reinterpret_cast<uint4*>(vpool + (row0 + n_old) * D + lig * EPV) = newkv[LPR + lig];
        if (lig == 0) { a.pos[row0 + n_old] = a.t; a.rnorm[row0 + n_old] = rn[new_li]; }
      } else {
        *reinterpret_cast<uint4*>(kpool + (row0 + n_old) * D + lig * EPV) = ld_global_v4(k_new + lig * EPV);
        *reinterpret_cast<uint4*>(vpool + (row0 + n_old) * D + lig * EPV) = ld_global_v4(v_new + lig * EPV);
      }
    }
    if (COMPRESS && rank == 0 && tid == 0) {
      a.len[sidx] = n;
      atomicAdd(&a.counters[kCntDecodeSteps], 1ull);
    }
    cluster_arrive();                                                // peers may still read our exchange area
    cluster_wait();
    return;
  }
  // ---- 4. victim (Eq. 7-8)
  unsigned long long kmin = ~0ull; int vic_rank = 0, vic_li = 0;
  for (int r = 0; r < C; ++r) {
    const Xch* x = cluster.map_shared_rank(xch, r);
    const unsigned long long t = x->cand_min;
    if (t < kmin) { kmin = t; vic_rank = r; vic_li = x->cand_min_li; }
  }
  if (kmin == ~0ull) {
    // nothing may be evicted (S_l < T + M): report, drop the new token, keep the cache as it is
    if (rank == 0 && tid == 0) report_error(a.status, D2O_ERR_STATE, 0xDEC00000u | (uint32_t)(sl & 0xfffff));
    cluster_arrive();
    cluster_wait();
    return;
  }
  const int vic_gi = vic_rank * chunk + vic_li;
  float kvic[EPV];
  float vic_rn;
  {
    const uint4* pks = cluster.map_shared_rank(ks, vic_rank);
    const uint4 kv = vic_li < a.res_rows ? pks[(size_t)vic_li * LPR + lig]
                                         : ld_global_v4((vic_gi < n_old ? kpool + (row0 + vic_gi) * D : k_new) + lig * EPV);
    Elem<T>::unpack(kv, kvic);
    vic_rn = cluster.map_shared_rank(rn, vic_rank)[vic_li];
  }
  // ---- 5. cosine similarity of the victim with every other row (Eq. 9), arg-max, ties -> earliest position
  {
    unsigned long long best = 0ull; int best_li = -1;
    for (int li = grp; li < cnt; li += NGRP) {
      if (r0 + li == vic_gi) continue;
      float f[EPV];
      const uint4 kv = li < a.res_rows ? ks[(size_t)li * LPR + lig] : ld_global_v4(k_src(li) + lig * EPV);
      Elem<T>::unpack(kv, f);
      float s = 0.f;
#pragma unroll
      for (int e = 0; e < EPV; ++e) s = fmaf(kvic[e], f[e], s);
      s = group_sum<LPR>(s, gmask);
      const float u = s * vic_rn * rn[li];
      const unsigned long long key = ((unsigned long long)float_ord(u) << 32) | (uint32_t)(0x7fffffff - ps[li]);
      if (key > best) { best = key; best_li = li; }
    }
    block_arg_extreme<false>(best, best_li, s_key, s_li, &xch->cand_max, &xch->cand_max_li);
  }
  cluster_arrive();                                                  // #3 neighbour candidates published
  cluster_wait();
  unsigned long long kmax = 0ull; int nn_rank = 0, nn_li = 0;
  for (int r = 0; r < C; ++r) {
    const Xch* x = cluster.map_shared_rank(xch, r);
    const unsigned long long t = x->cand_max;
    if (t > kmax) { kmax = t; nn_rank = r; nn_li = x->cand_max_li; }
  }
  const float mx = ord_float((uint32_t)(kmax >> 32));
  // ---- 6. EMA threshold (Eq. 10) and merge (Eq. 11-12)
  const float tau_new = a.beta * mx + (1.0f - a.beta) * tau_old;
  const float thr = isnan(a.tau_override) ? tau_new : a.tau_override;
  const bool merge = mx >= thr;
  if (rank == 0 && tid == 0) {
    a.tau[sidx] = tau_new;
    atomicAdd(&a.counters[kCntDecodeSteps], 1ull);
    atomicAdd(&a.counters[kCntEvictions], 1ull);
    atomicAdd(&a.counters[merge ? kCntMerges : kCntDiscards], 1ull);
  }
  if (merge && rank == nn_rank && grp == 0) {
    const int lj = nn_li;
    const bool is_new = (r0 + lj == n_old);
    const float ew = expf(mx);
    const float w_e = ew / (ew + kEuler), w_c = kEuler / (ew + kEuler);
    float fk[EPV], fv[EPV], vv[EPV];
    const uint4 kcur = is_new ? newkv[lig]
                              : (lj < a.res_rows ? ks[(size_t)lj * LPR + lig] : ld_global_v4(k_src(lj) + lig * EPV));
    Elem<T>::unpack(kcur, fk);
    Elem<T>::unpack(is_new ? newkv[LPR + lig] : ld_global_v4(v_src(lj) + lig * EPV), fv);
    // the victim's value row is still in place: its slot is overwritten only after the last barrier
    Elem<T>::unpack(ld_global_v4((vic_gi < n_old ? vpool + (row0 + vic_gi) * D : v_new) + lig * EPV), vv);
#pragma unroll
    for (int e = 0; e < EPV; ++e) { fk[e] = w_c * fk[e] + w_e * kvic[e]; fv[e] = w_c * fv[e] + w_e * vv[e]; }
    const uint4 kn = Elem<T>::pack(fk), vn = Elem<T>::pack(fv);
    Elem<T>::unpack(kn, fk);                                         // norm of what is stored
    float ss = 0.f;
#pragma unroll
    for (int e = 0; e < EPV; ++e) ss = fmaf(fk[e], fk[e], ss);
    ss = group_sum<LPR>(ss, gmask);
    const float rnew = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
    if (is_new) { newkv[lig] = kn; newkv[LPR + lig] = vn; }
    else {
      *reinterpret_cast<uint4*>(kpool + (row0 + r0 + lj) * D + lig * EPV) = kn;
      *reinterpret_cast<uint4*>(vpool + (row0 + r0 + lj) * D + lig * EPV) = vn;
      if (lig == 0) a.rnorm[row0 + r0 + lj] = rnew;
    }
    if (lig == 0) rn[lj] = rnew;
  }
  cluster_arrive();                                                  // #4 all reads of peer memory and of the victim's row are done
  cluster_wait();
  // ---- 7. the new token takes the victim's row
  if (rank == new_rank && vic_gi != n_old && grp == 0) {
    *reinterpret_cast<uint4*>(kpool + (row0 + vic_gi) * D + lig * EPV) = newkv[lig];
    *reinterpret_cast<uint4*>(vpool + (row0 + vic_gi) * D + lig * EPV) = newkv[LPR + lig];
    if (lig == 0) {
      a.pos[row0 + vic_gi] = a.t;
      a.score[row0 + vic_gi] = sc[new_li];
      a.rnorm[row0 + vic_gi] = rn[new_li];
    }
  }
}

// ------------------------------------------------------------------------------------ launch
template <typename T, int D, int G, bool COMPRESS>
static cudaError_t launch_one(const DecodeArgs& a, int n_slices, int C, const void* q, const void* k, const void* v,
                              void* out, void* kpool, void* vpool, cudaStream_t st) {
  constexpr int LPR = D * sizeof(T) / 16;
  const size_t smem = sizeof(Exchange<G, D>) + (size_t)kDecWarps * G * D * 4 + (size_t)(G + 3) * a.chunk_cap * 4 +
                      (size_t)2 * LPR * 16 + (size_t)a.res_rows * LPR * 16;
  auto kern = decode_kernel<T, D, G, COMPRESS>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(n_slices * C));
  cfg.blockDim = dim3(kDecThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, a, (const T*)q, (const T*)k, (const T*)v, (T*)out, (T*)kpool, (T*)vpool);
}

template <typename T, int D, bool COMPRESS>
static cudaError_t launch_g(int G, const DecodeArgs& a, int n_slices, int C, const void* q, const void* k,
                            const void* v, void* out, void* kpool, void* vpool, cudaStream_t st) {
  switch (G) {
    case 1: return launch_one<T, D, 1, COMPRESS>(a, n_slices, C, q, k, v, out, kpool, vpool, st);
    case 2: return launch_one<T, D, 2, COMPRESS>(a, n_slices, C, q, k, v, out, kpool, vpool, st);
    case 4: return launch_one<T, D, 4, COMPRESS>(a, n_slices, C, q, k, v, out, kpool, vpool, st);
    default: return launch_one<T, D, 8, COMPRESS>(a, n_slices, C, q, k, v, out, kpool, vpool, st);
  }
}

template <bool COMPRESS>
static cudaError_t launch_any(int dtype, int d, int G, const DecodeArgs& a, int n_slices, int C, const void* q,
                              const void* k, const void* v, void* out, void* kpool, void* vpool, cudaStream_t st) {
  if (dtype == D2O_F32)
    return d == 64 ? launch_g<float, 64, COMPRESS>(G, a, n_slices, C, q, k, v, out, kpool, vpool, st)
                   : launch_g<float, 128, COMPRESS>(G, a, n_slices, C, q, k, v, out, kpool, vpool, st);
  if (dtype == D2O_F16)
    return d == 64 ? launch_g<__half, 64, COMPRESS>(G, a, n_slices, C, q, k, v, out, kpool, vpool, st)
                   : launch_g<__half, 128, COMPRESS>(G, a, n_slices, C, q, k, v, out, kpool, vpool, st);
  return d == 64 ? launch_g<__nv_bfloat16, 64, COMPRESS>(G, a, n_slices, C, q, k, v, out, kpool, vpool, st)
                 : launch_g<__nv_bfloat16, 128, COMPRESS>(G, a, n_slices, C, q, k, v, out, kpool, vpool, st);
}

// Picks the cluster size and the shared-memory split for `max_rows` rows per slice.
static bool plan(int max_rows, int row_bytes, int G, int D, int want_cluster, bool resident, int n_slices, int* C_out,
                 int* chunk_cap, int* res_rows) {
  const int fixed = 2048 + G * D * 4 + kDecWarps * G * D * 4 + 1024;      // exchange area + reduction buffer + slack
  const int budget = 200 * 1024;
  int C = want_cluster;
  if (C == 0) {
    // smallest cluster that keeps all K rows resident in <= ~72 KB per CTA (three CTAs per SM), but enough CTAs
    // to cover the machine when there are few slices
    C = 1;
    while (C < kMaxCluster) {
      const int chunk = (((max_rows + C - 1) / C) + 7) & ~7;
      const long need = fixed + (long)chunk * ((G + 3) * 4 + (resident ? row_bytes : 0));
      if (need <= 72 * 1024 && (long)n_slices * C >= 2 * 148) break;
      C *= 2;
    }
  }
  const int chunk = (((max_rows + C - 1) / C) + 7) & ~7;
  long meta = fixed + (long)chunk * (G + 3) * 4;
  if (meta > budget) return false;
  long rr = resident ? (budget - meta) / row_bytes : 0;
  if (rr > chunk) rr = chunk;
  *C_out = C; *chunk_cap = chunk; *res_rows = (int)rr;
  return true;
}

cudaError_t launch_decode(const d2o_ctx* c, int l0, int l1, const void* q, const void* k, const void* v, void* out,
                          cudaStream_t st, d2o_status* why) {
  const d2o_config& g = c->cfg;
  const int B = g.batch, L = g.n_layers;
  DecodeArgs a = {};
  char* S = c->state;
  a.budgets = (const int32_t*)(S + c->lay.budgets);
  a.windows = (const int32_t*)(S + c->lay.windows);
  a.row_off = (const int64_t*)(S + c->lay.row_off);
  a.pos = (int32_t*)(S + c->lay.pos); a.score = (float*)(S + c->lay.score); a.rnorm = (float*)(S + c->lay.rnorm);
  a.len = (int32_t*)(S + c->lay.len); a.tau = (float*)(S + c->lay.tau);
  a.counters = (unsigned long long*)(S + c->lay.counters); a.status = (uint32_t*)(S + c->lay.status);
  a.L = L; a.l0 = l0; a.B = B; a.Hkv = g.n_kv_heads; a.T = g.n_sink;
  a.t = g.prompt_len + c->layer_steps[l0];
  a.beta = g.beta; a.tau_override = g.tau_override;
  int max_rows = 0;
  for (int l = l0; l < l1; ++l)
    for (int b = 0; b < B; ++b) {
      const int Sl = c->h_budgets[b * L + l];
      const int len = min(Sl, g.prompt_len + c->layer_steps[l0]);
      max_rows = max(max_rows, len + 1);
    }
  const int n_slices = (l1 - l0) * B * g.n_kv_heads;
  int C, chunk_cap, res_rows;
  if (!plan(max_rows, g.d_head * c->elem_size, c->group, g.d_head, c->decode_cluster, !c->decode_nonresident, n_slices,
            &C, &chunk_cap, &res_rows)) {
    *why = D2O_ERR_UNSUPPORTED;
    return cudaSuccess;
  }
  a.chunk_cap = chunk_cap; a.res_rows = res_rows;
  return launch_any<true>(g.dtype, g.d_head, c->group, a, n_slices, C, q, k, v, out, S + c->lay.kpool,
                          S + c->lay.vpool, st);
}

cudaError_t launch_full_decode(int dtype, int d, int n_slices, int group, int capacity, int len, void* kc, void* vc,
                               const void* q, const void* k, const void* v, void* out, cudaStream_t st,
                               d2o_status* why) {
  DecodeArgs a = {};
  a.full_capacity = capacity; a.full_len = len;
  int C, chunk_cap, res_rows;
  const int esz = dtype == D2O_F32 ? 4 : 2;
  if (!plan(len + 1, d * esz, group, d, 0, false, n_slices, &C, &chunk_cap, &res_rows)) {
    *why = D2O_ERR_UNSUPPORTED;
    return cudaSuccess;
  }
  a.chunk_cap = chunk_cap; a.res_rows = 0;
  return launch_any<false>(dtype, d, group, a, n_slices, C, q, k, v, out, kc, vc, st);
}

}  // namespace d2o
