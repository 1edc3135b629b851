// Column sums of the causal prompt attention (Section 4.1, Eq. 4; Eq. 6 case 1) for 16-bit Q/K on the
// 5th-generation tensor cores.  The P x P probability matrix is never stored: two sweeps recompute the
// logits tile by tile with tcgen05.mma (fp32 accumulators in tensor memory) and reduce them on the fly.
//
//   sweep 1 (rows)     lse2_i = log2 sum_{j<=i} 2^{c q_i.k_j},  c = log2(e)/sqrt(d)
//                      A = 256 query rows of one head (resident), B = key tiles 0 .. diagonal (streamed)
//   sweep 2 (columns)  s_j = sum_{i>=j} 2^{c q_i.k_j - lse2_i}
//                      A = 256 keys (resident), B = query tiles diagonal .. end (streamed, with their lse2)
// In both sweeps the quantity that is reduced belongs to an A row, i.e. to one tensor-memory lane, i.e.
// to one thread of the epilogue, and the reduction runs over that thread's registers: no shuffles, no
// atomics, a fixed order, bit-reproducible.  Across jobs the per-thread partials are added in fp64
// (sweep 2) so that a column which receives up to P probabilities keeps full fp32 accuracy.
//
// One CTA = (head, 256 A rows).  One job = one streamed tile of 128 B rows against both 128-row A
// tiles: two 128 x 128 x d MMAs whose accumulators fill one of two 256-column tensor-memory buffers.
//   warp 0      TMA producer (A once; B tiles and, in sweep 2, their lse2 through a 4-stage ring)
//   warp 1      tensor-memory allocation, MMA issue
//   warps 2-17  epilogue: four warps per quarter of the lanes; warp parts 0,1 take the first A tile
//               (B rows 0-63 / 64-127), parts 2,3 the second; exp2 on the MUFU pipe is what bounds a job
#include <math.h>

#include "d2o_common.cuh"
#include "d2o_tc.cuh"

namespace d2o {

constexpr int kCsEpiWarps = 16;
constexpr int kCsThreads = (2 + kCsEpiWarps) * 32;
constexpr int kCsTile = 128;                 // rows per MMA operand tile (M and N)
constexpr int kCsStages = 4;                 // B ring
enum { kSweepRows = 0, kSweepCols = 1 };

struct ColsumTcArgs {
  float* lse2;                               // [B, Hq, P] log2-domain row normalisers (written by sweep 1, read by sweep 2)
  float* colsum;                             // [B, Hq, P] (sweep 2)
  uint32_t* status;
  const int32_t* plen;                       // [B] prompt length of every sequence (<= P)
  int P, Hq, group;                          // P: the length the tensors are laid out for
};

namespace tc {
// global -> this CTA's shared memory, 16-byte aligned on both sides, size a multiple of 16
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// 2^x on the special-function unit (one instruction; results below 2^-126 flush to zero)
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// maximum of three; a NaN operand is ignored
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
}  // namespace tc

template <int D, int FMT, int SWEEP>
__global__ void __launch_bounds__(kCsThreads, 1)
attn_tc_kernel(ColsumTcArgs a, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k) {
  constexpr int KB = D / 64;                                 // 64-element (128-byte) blocks along d
  constexpr int BLOCK = kCsTile * 128;                       // bytes of one k-block of one 128-row tile
  constexpr int TILE = KB * BLOCK;                           // bytes of one 128-row tile
  constexpr uint32_t IDESC = make_idesc(FMT, kCsTile, kCsTile);
  const float c = (D == 64 ? 0.125f : 0.08838834764831845f) * kLog2e;

  extern __shared__ __align__(1024) unsigned char cs_smem[];
  unsigned char* sA = cs_smem;                               // [2 tiles][KB][128 rows][128 B]
  unsigned char* sB = cs_smem + 2 * TILE;                    // [stages][KB][128 rows][128 B]
  float* s_lse = reinterpret_cast<float*>(sB + kCsStages * TILE);   // [stages][128] lse2 of the B rows (sweep 2)
  float* s_comb = s_lse + kCsStages * kCsTile;               // [2][2][128] partner values for the final combination
  __shared__ unsigned long long a_full, b_full[kCsStages], b_empty[kCsStages], tm_full[2], tm_empty[2];
  __shared__ uint32_t s_tmem;
  __shared__ int s_fail;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int bh = blockIdx.x;                                 // b * Hq + hq (fastest index: all heads of the heaviest pair first)
  const int b = bh / a.Hq, hq = bh % a.Hq;
  const int P = a.plen[b];                                   // this sequence's prompt; rows beyond it are padding
  const int n_pairs = (P + 2 * kCsTile - 1) / (2 * kCsTile);
  const int n_tiles = (P + kCsTile - 1) / kCsTile;
  if ((int)blockIdx.y >= n_pairs) return;                    // the grid is sized for the longest prompt
  const int Hkv = a.Hq / a.group;
  const int q_base = bh * a.P;                               // first row of this head in the [B*Hq*P, d] view of Q
  const int k_base = (b * Hkv + hq / a.group) * a.P;
  // heaviest CTAs first: sweep 1 -> the last rows see the most keys; sweep 2 -> the first keys see the most rows
  const int pair = SWEEP == kSweepRows ? n_pairs - 1 - (int)blockIdx.y : (int)blockIdx.y;
  const int a0 = pair * 2 * kCsTile;                         // first A row (query position or key position)
  // streamed tiles: sweep 1 keys [0, a0 + 256), sweep 2 queries [a0, P)
  const int bt0 = SWEEP == kSweepRows ? 0 : a0 / kCsTile;
  const int bt1 = SWEEP == kSweepRows ? min(n_tiles, (a0 + 2 * kCsTile) / kCsTile) : n_tiles;
  const int n_jobs = bt1 - bt0;
  if ((tc::smem_u32(cs_smem) & 1023u) != 0u) {               // swizzled tiles need 1024-byte aligned shared memory
    if (tid == 0) report_error(a.status, D2O_ERR_STATE, 0xC5C10000u);
    return;
  }

  if (tid == 0) {
    s_fail = 0;
    tc::mbar_init(&a_full, 1);
    for (int s = 0; s < kCsStages; ++s) { tc::mbar_init(&b_full[s], 1); tc::mbar_init(&b_empty[s], 1 + kCsEpiWarps); }
    for (int i = 0; i < 2; ++i) { tc::mbar_init(&tm_full[i], 1); tc::mbar_init(&tm_empty[i], kCsEpiWarps); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {                                           // 512 columns: two buffers of 2 x (128 x 128) fp32
    tc::tmem_alloc(&s_tmem, 512);
    tc::tmem_relinquish();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem_base = s_tmem;

  if (warp == 0) {
    // ======================================================================= TMA producer
    if (lane == 0) {
      const CUtensorMap* map_a = SWEEP == kSweepRows ? &map_q : &map_k;
      const CUtensorMap* map_b = SWEEP == kSweepRows ? &map_k : &map_q;
      const int a_base = SWEEP == kSweepRows ? q_base : k_base;
      const int b_base = SWEEP == kSweepRows ? k_base : q_base;
      tc::mbar_expect_tx(&a_full, (uint32_t)(2 * TILE));
      for (int t = 0; t < 2; ++t)
        for (int kb = 0; kb < KB; ++kb)
          tc::tma_load_2d(sA + t * TILE + kb * BLOCK, map_a, kb * 64, a_base + a0 + t * kCsTile, &a_full);
      for (int job = 0; job < n_jobs; ++job) {
        const int s = job % kCsStages;
        if (job >= kCsStages && !s_fail && !tc::mbar_wait(&b_empty[s], (uint32_t)(((job / kCsStages) - 1) & 1))) s_fail = 1;
        const int r0 = (bt0 + job) * kCsTile;                // first B row of the tile
        uint32_t bytes = (uint32_t)TILE;
        // 16-byte granules: up to three entries past the prompt come from the row's padding and are masked
        const int n_lse = SWEEP == kSweepCols ? min(kCsTile, ((P + 3) & ~3) - r0) : 0;
        bytes += (uint32_t)(n_lse * 4);
        tc::mbar_expect_tx(&b_full[s], bytes);
        for (int kb = 0; kb < KB; ++kb)
          tc::tma_load_2d(sB + s * TILE + kb * BLOCK, map_b, kb * 64, b_base + r0, &b_full[s]);
        if (n_lse > 0) tc::bulk_g2s(s_lse + s * kCsTile, a.lse2 + (size_t)bh * a.P + r0, (uint32_t)(n_lse * 4), &b_full[s]);
      }
    }
  } else if (warp == 1) {
    // ======================================================================= MMA issuer
    if (lane == 0) {
      if (!tc::mbar_wait(&a_full, 0)) s_fail = 1;
      for (int job = 0; job < n_jobs; ++job) {
        const int s = job % kCsStages, buf = job & 1;
        if (!s_fail && !tc::mbar_wait(&b_full[s], (uint32_t)((job / kCsStages) & 1))) s_fail = 1;
        // the epilogue must have drained this buffer (the first use of each buffer passes at once)
        if (!s_fail && !tc::mbar_wait(&tm_empty[buf], (uint32_t)(((job >> 1) & 1) ^ 1))) s_fail = 1;
        tc::fence_after_sync();
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 256 + t * kCsTile);
#pragma unroll
          for (int kb = 0; kb < KB; ++kb) {
            const uint64_t adesc = tc::smem_desc_sw128(tc::smem_u32(sA + t * TILE + kb * BLOCK));
            const uint64_t bdesc = tc::smem_desc_sw128(tc::smem_u32(sB + s * TILE + kb * BLOCK));
#pragma unroll
            for (int k = 0; k < 4; ++k)                      // 16 elements = 32 bytes along d per instruction
              tc::mma_f16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), IDESC, (kb | k) != 0 ? 1u : 0u);
          }
        }
        tc::mma_commit(&tm_full[buf]);
        tc::mma_commit(&b_empty[s]);                         // one of the 17 arrivals that free the stage
      }
    }
  } else {
    // ======================================================================= epilogue warps
    const int e = warp - 2;
    const int quarter = warp & 3;                            // tensor-memory lanes this warp may read: 32*quarter ..
    const int part = e >> 2;                                 // 0,1: first A tile, B rows 0-63 / 64-127; 2,3: second A tile
    const int at = part >> 1, bhalf = part & 1;
    const int arow = a0 + at * kCsTile + quarter * 32 + lane;    // position of this thread's A row (query or key)
    // sweep 1: running maximum of the raw logits and sum of 2^{c (s - m)}; sweep 2: column sum
    float m_run = -INFINITY, l_run = 0.f;
    double col_acc = 0.0;
    uint32_t ra[32], rb[32];
#pragma unroll 1
    for (int job = 0; job < n_jobs; ++job) {
      const int s = job % kCsStages, buf = job & 1;
      const int brow0 = (bt0 + job) * kCsTile + bhalf * 64;   // position of the first B row this warp looks at
      if (!s_fail && !tc::mbar_wait(&tm_full[buf], (uint32_t)((job >> 1) & 1))) s_fail = 1;
      tc::fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * 256 + at * kCsTile + bhalf * 64);
      tc::tmem_ld32_issue(taddr, ra);
      tc::tmem_ld32_issue(taddr + 32u, rb);
      tc::tmem_ld_wait(ra);
      tc::tmem_ld_wait(rb);
      // both blocks are in registers: hand the accumulator back to the MMA warp
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&tm_empty[buf]);
      if (SWEEP == kSweepRows) {
        // B rows are keys: valid iff key <= query (keys >= P are > every stored query)
        const bool need_mask = brow0 + 63 > a0 + at * kCsTile + quarter * 32;     // warp-uniform
        // four independent chains of three-input maxima: the block maximum is on every thread's critical path
        float bmx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float x = __uint_as_float(ra[i]), y = __uint_as_float(rb[i]);
          if (need_mask) {
            if (brow0 + i > arow) x = -INFINITY;
            if (brow0 + 32 + i > arow) y = -INFINITY;
            ra[i] = __float_as_uint(x); rb[i] = __float_as_uint(y);
          }
          bmx[i & 3] = tc::max3(bmx[i & 3], x, y);
        }
        const float bm = fmaxf(fmaxf(bmx[0], bmx[1]), fmaxf(bmx[2], bmx[3]));
        if (bm > m_run) { l_run *= exp2f((m_run - bm) * c); m_run = bm; }      // exp2f(-inf) = 0 on the first block
        if (m_run > -INFINITY) {
          const float mc = m_run * c;
          float l0 = 0.f, l1 = 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            l0 += tc::ex2(fmaf(__uint_as_float(ra[i]), c, -mc));
            l1 += tc::ex2(fmaf(__uint_as_float(rb[i]), c, -mc));
          }
          l_run += l0 + l1;
        }
      } else {
        // B rows are queries: valid iff query >= key and query < P
        const float* ls = s_lse + s * kCsTile + bhalf * 64;
        const bool need_mask = (brow0 < a0 + at * kCsTile + quarter * 32 + 32) || (brow0 + 64 > P);   // warp-uniform
        float p0 = 0.f, p1 = 0.f;
        const float4* l4 = reinterpret_cast<const float4*>(ls);
#pragma unroll
        for (int i4 = 0; i4 < 8; ++i4) {
          const float4 la = l4[i4], lb = l4[8 + i4];
          const float lav[4] = {la.x, la.y, la.z, la.w}, lbv[4] = {lb.x, lb.y, lb.z, lb.w};
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            const int i = i4 * 4 + w;
            float x = tc::ex2(fmaf(__uint_as_float(ra[i]), c, -lav[w]));
            float y = tc::ex2(fmaf(__uint_as_float(rb[i]), c, -lbv[w]));
            if (need_mask) {
              const int qa = brow0 + i, qb = brow0 + 32 + i;
              if (qa < arow || qa >= P) x = 0.f;
              if (qb < arow || qb >= P) y = 0.f;
            }
            p0 += x; p1 += y;
          }
        }
        col_acc += (double)(p0 + p1);
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(&b_empty[s]);         // this warp is done with the stage's lse2
      }
      if (SWEEP == kSweepRows) {
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(&b_empty[s]);
      }
    }
    // combine the two warps that share an A row (B-row halves), fixed order
    const int r = quarter * 32 + lane;
    if (SWEEP == kSweepRows) {
      if (bhalf == 1) { s_comb[(at * 2 + 0) * kCsTile + r] = m_run; s_comb[(at * 2 + 1) * kCsTile + r] = l_run; }
      asm volatile("bar.sync 1, %0;" ::"n"(kCsEpiWarps * 32) : "memory");
      if (bhalf == 0 && arow < P) {
        const float m2 = s_comb[(at * 2 + 0) * kCsTile + r], l2 = s_comb[(at * 2 + 1) * kCsTile + r];
        const float mm = fmaxf(m_run, m2);
        const float ll = (m_run > -INFINITY ? l_run * exp2f((m_run - mm) * c) : 0.f) +
                         (m2 > -INFINITY ? l2 * exp2f((m2 - mm) * c) : 0.f);
        a.lse2[(size_t)bh * a.P + arow] = fmaf(mm, c, log2f(ll));
      }
    } else {
      double* dcomb = reinterpret_cast<double*>(s_comb);
      if (bhalf == 1) dcomb[at * kCsTile + r] = col_acc;
      asm volatile("bar.sync 1, %0;" ::"n"(kCsEpiWarps * 32) : "memory");
      if (bhalf == 0 && arow < P) a.colsum[(size_t)bh * a.P + arow] = (float)(col_acc + dcomb[at * kCsTile + r]);
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc::fence_after_sync();
    tc::tmem_dealloc(tmem_base, 512);
  }
  if (tid == 0 && s_fail) report_error(a.status, D2O_ERR_TIMEOUT, 0xC5C00000u | (uint32_t)(bh & 0xfffff));
}

// natural-log row normalisers supplied by the caller -> log2 domain
__global__ void lse_to_log2_kernel(const float* __restrict__ lse, float* __restrict__ lse2, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) lse2[i] = lse[i] * kLog2e;
}

bool colsum_tc_supported(const d2o_config* cfg) {
  return cfg->dtype != D2O_F32 && cfg->prompt_len % 4 == 0;
}

// Column sums of one layer on the tensor cores.  `lse_in` (natural log, may be NULL) replaces sweep 1.
cudaError_t launch_colsum_tc(const d2o_ctx* c, const void* Q, const void* K, const float* lse_in, float* colsum,
                             cudaStream_t st, int lane) {
  const d2o_config& g = c->cfg;
  const int B = g.batch, Hq = g.n_q_heads, Hkv = g.n_kv_heads, P = g.prompt_len, D = g.d_head;
  CUtensorMap map_q, map_k;
  if (!encode_rows_2d(&map_q, g.dtype, Q, (uint64_t)B * Hq * P, D, kCsTile)) return cudaErrorNotSupported;
  if (!encode_rows_2d(&map_k, g.dtype, K, (uint64_t)B * Hkv * P, D, kCsTile)) return cudaErrorNotSupported;
  ColsumTcArgs a;
  a.lse2 = (float*)(c->scratch + c->slay.lse + (size_t)lane * c->slay.lse_stride);
  a.colsum = colsum;
  a.status = (uint32_t*)(c->state + c->lay.status);
  a.P = P; a.Hq = Hq; a.group = c->group;
  a.plen = (const int32_t*)(c->state + c->lay.plen);
  const int KB = D / 64;
  const size_t smem = (size_t)(2 + kCsStages) * KB * kCsTile * 128 + (size_t)kCsStages * kCsTile * 4 + 4 * kCsTile * 4;
  const int n_pairs = (P + 2 * kCsTile - 1) / (2 * kCsTile);
  // heaviest CTAs first over the whole launch: the pair index is the slow grid dimension
  dim3 grid(B * Hq, n_pairs);
  const int fmt = g.dtype == D2O_F16 ? 0 : 1;
  cudaError_t e;
#define D2O_LAUNCH_CS(DD, FF, SW)                                                                                  \
  do {                                                                                                             \
    e = cudaFuncSetAttribute(attn_tc_kernel<DD, FF, SW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
    if (e != cudaSuccess) return e;                                                                                \
    attn_tc_kernel<DD, FF, SW><<<grid, kCsThreads, smem, st>>>(a, map_q, map_k);                                   \
  } while (0)
#define D2O_LAUNCH_CS_ALL(SW)                                                                    \
  do {                                                                                           \
    if (D == 128) { if (fmt == 0) D2O_LAUNCH_CS(128, 0, SW); else D2O_LAUNCH_CS(128, 1, SW); }   \
    else          { if (fmt == 0) D2O_LAUNCH_CS(64, 0, SW); else D2O_LAUNCH_CS(64, 1, SW); }     \
  } while (0)
  if (lse_in) {
    const size_t n = (size_t)B * Hq * P;
    lse_to_log2_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(lse_in, a.lse2, n);
  } else {
    D2O_LAUNCH_CS_ALL(kSweepRows);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  D2O_LAUNCH_CS_ALL(kSweepCols);
#undef D2O_LAUNCH_CS_ALL
#undef D2O_LAUNCH_CS
  return cudaGetLastError();
}

}  // namespace d2o
