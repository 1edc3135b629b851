// Uncompressed decode attention (Section 3, Eq. 2-3): the comparison kernel for the compressed path.
//
// One thread-block cluster handles one slice = (sequence, KV head) with its G query heads; the
// len+1 rows (cache + the new token) are split evenly over the CTAs of the cluster.  Each CTA
// streams its K rows once (logits), publishes its softmax (max, sum), streams its V rows once
// (un-normalised outputs) and rank 0 combines the partial outputs through distributed shared
// memory.  The new token's row is appended at row `len`.
#include <cooperative_groups.h>
#include <math.h>

#include "d2o_common.cuh"

namespace cg = cooperative_groups;

namespace d2o {

constexpr int kFullThreads = 256;
constexpr int kFullWarps = kFullThreads / 32;
constexpr int kFullMaxCluster = 8;

struct FullArgs {
  int capacity, len;
  int chunk_cap;                    // rows per CTA the shared-memory arrays are sized for
};

template <int G, int D>
struct alignas(16) FullExchange {    // the part of shared memory that peer CTAs read
  float m[G];
  float l[G];
  float acc[G][D];
};

template <typename T, int D, int G>
__global__ void __launch_bounds__(kFullThreads, (G <= 2 ? 3 : 2))
full_decode_kernel(FullArgs a, const T* __restrict__ q_in, const T* __restrict__ k_in, const T* __restrict__ v_in,
                   T* __restrict__ out, T* __restrict__ kcache, T* __restrict__ vcache) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int LPR = D / EPV;                  // lanes that share one row (16-byte segment each)
  constexpr int NGRP = kFullThreads / LPR;      // rows in flight per CTA iteration
  using Xch = FullExchange<G, D>;

  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int sl = blockIdx.x / C;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int grp = tid / LPR, lig = tid % LPR;
  const unsigned gmask = group_mask<LPR>();

  const int64_t row0 = (int64_t)sl * a.capacity;
  const int n_old = a.len;
  const int n = n_old + 1;
  const int chunk = (((n + C - 1) / C) + 7) & ~7;
  const int r0 = rank * chunk;
  const int cnt = max(0, min(n, r0 + chunk) - r0);

  extern __shared__ __align__(16) unsigned char dsm[];
  Xch* xch = reinterpret_cast<Xch*>(dsm);
  float* red = reinterpret_cast<float*>(dsm + sizeof(Xch));        // [warps][G][D]
  float* pl = red + kFullWarps * G * D;                             // [G][chunk_cap] logits -> probabilities
  __shared__ float s_red[kFullWarps][G];

  const T* k_new = k_in + (size_t)sl * D;
  const T* v_new = v_in + (size_t)sl * D;
  auto k_src = [&](int li) -> const T* {
    const int gi = r0 + li;
    return gi < n_old ? kcache + (row0 + gi) * D : k_new;
  };
  auto v_src = [&](int li) -> const T* {
    const int gi = r0 + li;
    return gi < n_old ? vcache + (row0 + gi) * D : v_new;
  };

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
  // ---- K pass: logits
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
        float f[EPV];
        Elem<T>::unpack(kv[u], f);
        float dot[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float s = 0.f;
#pragma unroll
          for (int e = 0; e < EPV; ++e) s = fmaf(qf[g][e], f[e], s);
          dot[g] = group_sum<LPR>(s, gmask);
        }
        if (lig == 0) {
#pragma unroll
          for (int g = 0; g < G; ++g) pl[(size_t)g * a.chunk_cap + li] = dot[g];
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
    for (int li = tid; li < cnt; li += kFullThreads) {
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
      for (int w = 1; w < kFullWarps; ++w) t = fmaxf(t, s_red[w][g]);
      m_loc[g] = t;
    }
    __syncthreads();
    float sum[G];
#pragma unroll
    for (int g = 0; g < G; ++g) sum[g] = 0.f;
    for (int li = tid; li < cnt; li += kFullThreads) {
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
      for (int w = 0; w < kFullWarps; ++w) t += s_red[w][g];
      l_loc[g] = t;
    }
#pragma unroll
    for (int g = 0; g < G; ++g)
      if (tid == g) { xch->m[g] = m_loc[g]; xch->l[g] = l_loc[g]; }
  }
  // ---- V pass: un-normalised outputs
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
        }
      }
    }
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
    for (int i = tid; i < G * D; i += kFullThreads) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < kFullWarps; ++w) t += red[(size_t)w * G * D + i];
      xch->acc[i / D][i % D] = t;
    }
  }
  cluster.sync();                                                    // (max, sum, partial outputs) of every CTA are visible
  if (rank == 0) {
    for (int i = tid; i < G * D; i += kFullThreads) {
      const int g = i / D, dd = i % D;
      float ms = -INFINITY;
      for (int r = 0; r < C; ++r) ms = fmaxf(ms, cluster.map_shared_rank(xch, r)->m[g]);
      float ls = 0.f, num = 0.f;
      for (int r = 0; r < C; ++r) {
        const Xch* x = cluster.map_shared_rank(xch, r);
        const float w = exp2f(x->m[g] - ms);
        ls = fmaf(x->l[g], w, ls);
        num = fmaf(x->acc[g][dd], w, num);
      }
      out[((size_t)sl * G + g) * D + dd] = Elem<T>::from_float(num / ls);
    }
  }
  // append the new token's row
  if (rank == n_old / chunk && grp == 0) {
    *reinterpret_cast<uint4*>(kcache + (row0 + n_old) * D + lig * EPV) = ld_global_v4(k_new + lig * EPV);
    *reinterpret_cast<uint4*>(vcache + (row0 + n_old) * D + lig * EPV) = ld_global_v4(v_new + lig * EPV);
  }
  cluster.sync();                                                    // rank 0 may still read our exchange area
}

// ------------------------------------------------------------------------------------ launch
template <typename T, int D, int G>
static cudaError_t launch_one(const FullArgs& a, int n_slices, int C, const void* q, const void* k, const void* v,
                              void* out, void* kc, void* vc, cudaStream_t st) {
  const size_t smem = sizeof(FullExchange<G, D>) + (size_t)kFullWarps * G * D * 4 + (size_t)G * a.chunk_cap * 4;
  auto kern = full_decode_kernel<T, D, G>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(n_slices * C));
  cfg.blockDim = dim3(kFullThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, a, (const T*)q, (const T*)k, (const T*)v, (T*)out, (T*)kc, (T*)vc);
}

template <typename T, int D>
static cudaError_t launch_g(int G, const FullArgs& a, int n_slices, int C, const void* q, const void* k,
                            const void* v, void* out, void* kc, void* vc, cudaStream_t st) {
  switch (G) {
    case 1: return launch_one<T, D, 1>(a, n_slices, C, q, k, v, out, kc, vc, st);
    case 2: return launch_one<T, D, 2>(a, n_slices, C, q, k, v, out, kc, vc, st);
    case 4: return launch_one<T, D, 4>(a, n_slices, C, q, k, v, out, kc, vc, st);
    default: return launch_one<T, D, 8>(a, n_slices, C, q, k, v, out, kc, vc, st);
  }
}

cudaError_t launch_full_decode(int dtype, int d, int n_slices, int group, int capacity, int len, void* kc, void* vc,
                               const void* q, const void* k, const void* v, void* out, cudaStream_t st,
                               d2o_status* why) {
  FullArgs a = {};
  a.capacity = capacity; a.len = len;
  // smallest cluster that gives the machine two waves of CTAs and keeps the logits of a CTA under 64 KB
  int C = 1;
  const int rows = len + 1;
  int sms = 0, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return cudaGetLastError();
  while (C < kFullMaxCluster) {
    const int chunk = (((rows + C - 1) / C) + 7) & ~7;
    if ((long)chunk * group * 4 <= 64 * 1024 && (long)n_slices * C >= 2L * sms) break;
    C *= 2;
  }
  a.chunk_cap = (((rows + C - 1) / C) + 7) & ~7;
  if ((long)a.chunk_cap * group * 4 > 160 * 1024) { *why = D2O_ERR_UNSUPPORTED; return cudaSuccess; }
  if (dtype == D2O_F32)
    return d == 64 ? launch_g<float, 64>(group, a, n_slices, C, q, k, v, out, kc, vc, st)
                   : launch_g<float, 128>(group, a, n_slices, C, q, k, v, out, kc, vc, st);
  if (dtype == D2O_F16)
    return d == 64 ? launch_g<__half, 64>(group, a, n_slices, C, q, k, v, out, kc, vc, st)
                   : launch_g<__half, 128>(group, a, n_slices, C, q, k, v, out, kc, vc, st);
  return d == 64 ? launch_g<__nv_bfloat16, 64>(group, a, n_slices, C, q, k, v, out, kc, vc, st)
                 : launch_g<__nv_bfloat16, 128>(group, a, n_slices, C, q, k, v, out, kc, vc, st);
}

}  // namespace d2o
