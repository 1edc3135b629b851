// Nearest-neighbour matching at the prompt stage (Section 4.2, Eq. 9) for 16-bit keys on the
// 5th-generation tensor cores: U = K_e K_c^T as tcgen05.mma (kind::f16, fp32 accumulators in tensor
// memory), fused with the scaling by the inverse key norms and the row max / arg-max.
//
// The evicted keys are most of the prompt (80 - 95 % at the cache ratios of interest), in prompt
// order.  Instead of gathering them, the kernel multiplies ALL prompt rows of a slice with the
// retained keys and lets the consumer pick the evicted positions: the A operand is then a plain
// tiled TMA load of 128 consecutive prompt rows, and the few retained rows among them cost
// S/P extra work.
//
// One CTA = one work item = (slice, chunk of up to 384 retained rows, range of 128-row prompt tiles); the host
// cuts every (slice, chunk) into ranges of about equal work once the budgets are known (sim_tc_build_items).
//   warp 0      TMA producer: the retained chunk once (B operand, stays in shared memory), then the prompt tiles
//               (A operand) into four slots, one per part; 128-byte swizzled K-major tiles
//   warp 1      allocates tensor memory, issues tcgen05.mma: one job = 128 x 128 x d (d/16 instructions) into the
//               part's own 128-column accumulator, the parts in turn
//   warps 2-17  epilogue: four parts of four warps.  A part owns every fourth prompt tile; each of its threads owns
//               one row (tensor-memory lane) of that tile and scans all retained columns of it, job after job:
//               tcgen05.ld of the accumulator, times 1/|k_c| per column, running max and arg-max (ties -> lowest
//               slot) in registers.  No exchange between warps and no barrier per tile; while one part drains its
//               accumulator the tensor cores work for the other three.
// Output: for every prompt position of the tile range and this chunk, the packed key
// (ordered max_j k_i.k_j/|k_j|, 0x7fffffff - slot).  neighbour_reduce_kernel takes the maximum over
// the chunks at the evicted positions and multiplies by 1/|k_i|.
#include <cuda.h>
#include <limits.h>
#include <math.h>
#include <stdlib.h>

#include <algorithm>
#include <utility>
#include <vector>

#include "d2o_common.cuh"
#include "d2o_tc.cuh"

namespace d2o {

constexpr int kTcEpiWarps = 16;             // four per quarter of the tensor-memory lanes
constexpr int kTcThreads = (2 + kTcEpiWarps) * 32;
constexpr int kTileM = 128;                 // prompt rows per A tile
constexpr int kJobN = 128;                  // retained rows per MMA job (one 128 x 128 fp32 accumulator)
constexpr int kChunkN = 384;                // retained rows resident per CTA (96 KB for d = 128)
constexpr int kBBoxRows = 64;               // rows per TMA box of the B operand
constexpr int kParts = 4;                   // prompt tiles in flight: each with its own accumulator and four epilogue warps

struct SimTcArgs {
  const int32_t* budgets; const int64_t* row_off;
  const float* rnorm;                       // pool-wide 1/|k_c|
  unsigned long long* part_key;             // [slices][n_chunks_max][P]
  uint32_t* status;
  const int32_t* plen;                      // [B] prompt length of every sequence; P is the row stride per slice
  const int4* items;                        // work list of this layer: (slice, chunk, first tile, end tile) per CTA
  int L, layer, Hkv, P, n_chunks_max;
};

// Retained rows per chunk for a slice of S rows: ceil(S / kChunkN) chunks of equal size, rounded up to the MMA's
// column granularity.
__host__ __device__ __forceinline__ int chunk_columns(int S) {
  const int n_chunks = (S + kChunkN - 1) / kChunkN;
  return (((S + n_chunks - 1) / n_chunks) + 15) & ~15;
}

// (x0, x1) = (a0 * b0, a1 * b1), each product rounded to nearest as a single multiply would.
__device__ __forceinline__ void mul_pair(float a0, float a1, float b0, float b1, float& x0, float& x1) {
  unsigned long long a, b, d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(a) : "f"(a0), "f"(a1));
  asm("mov.b64 %0, {%1, %2};" : "=l"(b) : "f"(b0), "f"(b1));
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  asm("mov.b64 {%0, %1}, %2;" : "=f"(x0), "=f"(x1) : "l"(d));
}

// Maximum of three; a NaN operand is ignored.
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// One block of 32 accumulator columns of one row: times 1/|k_c| per column, maximum and its column (the lowest
// on ties), merged into the row's running (best, best_col).  cl0 = chunk-local column of the block.
__device__ __forceinline__ void scan_block(const uint32_t (&r)[32], const float* s_rn, int cl0, int n_cols, int c0,
                                           float& best, int& best_col) {
  const float4* rn4 = reinterpret_cast<const float4*>(s_rn + cl0);
  if (cl0 + 32 <= n_cols) {
    // Columns go in pairs (2i, 2i + 1): one packed multiply, one three-input maximum against the running value,
    // one compare and two selects per pair.  The chain remembers the winning pair and that pair's first value,
    // from which the column inside the pair follows at the end.  Two chains (pairs i mod 2) keep them short.
    // max.f32 drops a NaN operand, as the compare of the scalar form does.
    float pb[2] = {-INFINITY, -INFINITY}, plo[2] = {-INFINITY, -INFINITY};
    int pi[2] = {0, 1};
#pragma unroll
    for (int i4 = 0; i4 < 8; ++i4) {
      const float4 q = rn4[i4];
      const float rv[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int w = 0; w < 2; ++w) {
        float x0, x1;
        mul_pair(__uint_as_float(r[i4 * 4 + 2 * w]), __uint_as_float(r[i4 * 4 + 2 * w + 1]), rv[2 * w], rv[2 * w + 1], x0, x1);
        const float m = max3(pb[w], x0, x1);
        const bool up = m > pb[w];
        pi[w] = up ? i4 * 2 + w : pi[w];
        plo[w] = up ? x0 : plo[w];
        pb[w] = m;
      }
    }
    // the later chain wins only with a larger value or an equal one from an earlier pair
    if (pb[1] > pb[0] || (pb[1] == pb[0] && pi[1] < pi[0])) { pb[0] = pb[1]; pi[0] = pi[1]; plo[0] = plo[1]; }
    const int col = 2 * pi[0] + (plo[0] == pb[0] ? 0 : 1);        // equal values inside the pair: the lower column
    if (pb[0] > best) { best = pb[0]; best_col = c0 + cl0 + col; }
    return;
  }
  // four interleaved running maxima (columns i mod 4) keep the compare chains short
  float tb[4]; int ti[4];
#pragma unroll
  for (int w = 0; w < 4; ++w) { tb[w] = -INFINITY; ti[w] = w; }
  {                                                               // columns past the chunk hold other slices' rows
#pragma unroll
    for (int i4 = 0; i4 < 8; ++i4) {
      const float4 q = rn4[i4];
      const float rv[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const float x = __uint_as_float(r[i4 * 4 + w]) * rv[w];
        if (cl0 + i4 * 4 + w < n_cols && x > tb[w]) { tb[w] = x; ti[w] = i4 * 4 + w; }
      }
    }
  }
  // larger value wins, equal values go to the lower column
#pragma unroll
  for (int w = 1; w < 4; ++w)
    if (tb[w] > tb[0] || (tb[w] == tb[0] && ti[w] < ti[0])) { tb[0] = tb[w]; ti[0] = ti[w]; }
  if (tb[0] > best) { best = tb[0]; best_col = c0 + cl0 + ti[0]; }   // ascending blocks: the first maximum stays
}

template <int D, int FMT>
__global__ void __launch_bounds__(kTcThreads, 1)
sim_tc_kernel(SimTcArgs a, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_pool) {
  constexpr int KB = D / 64;                                 // 64-element (128-byte) blocks along d
  constexpr int A_BLOCK = kTileM * 128;                      // bytes of one A k-block
  constexpr int A_TILE = KB * A_BLOCK;
  constexpr int B_BLOCK = kChunkN * 128;                     // bytes of one B k-block (all chunk rows)

  extern __shared__ __align__(1024) unsigned char tc_smem[];
  unsigned char* sB = tc_smem;                               // [KB][kChunkN rows][128 B]
  unsigned char* sA = tc_smem + KB * B_BLOCK;                // [kParts][KB][128 rows][128 B]: the prompt tile of each part
  float* s_rn = reinterpret_cast<float*>(sA + kParts * A_TILE);                    // [kChunkN] 1/|k_c| of the chunk
  __shared__ unsigned long long b_full, a_full[kParts], a_empty[kParts], tm_full[kParts], tm_empty[kParts];
  __shared__ uint32_t s_tmem;
  __shared__ int s_fail;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int4 item = a.items[blockIdx.x];
  const int slice = item.x;
  const int nc = item.y;
  const int b = slice / a.Hkv, h = slice % a.Hkv;
  const int S = a.budgets[slice_entry(b, a.layer, h, a.L, a.Hkv)];
  const int chunk_cols = chunk_columns(S);                   // the retained rows are split evenly over the chunks
  const int c0 = nc * chunk_cols;                            // first retained slot of the chunk
  const int Pb = a.plen[b];                                  // this sequence's prompt length
  if (c0 >= S || Pb - S <= 0) return;                        // uniform for the CTA: nothing to do
  const int n_cols = min(chunk_cols, S - c0);
  const int n_j = (n_cols + kJobN - 1) / kJobN;              // MMA column tiles (jobs) per prompt tile: 1 .. 3
  const int n_last = (n_cols - (n_j - 1) * kJobN + 15) & ~15;    // columns of the last job's MMA (multiple of 16)
  const int n_tiles_all = (Pb + kTileM - 1) / kTileM;
  const int t0 = item.z;
  const int t1 = min(n_tiles_all, item.w);
  if (t0 >= t1) return;
  const int T = t1 - t0;                                     // prompt tiles of this CTA; part p takes tiles p, p + 4, ...
  const int64_t row0 = a.row_off[slice_entry(b, a.layer, h, a.L, a.Hkv)];
  if ((tc::smem_u32(tc_smem) & 1023u) != 0u) {               // swizzled tiles need 1024-byte aligned shared memory
    if (tid == 0) report_error(a.status, D2O_ERR_STATE, 0x51C10000u);
    return;
  }

  if (tid == 0) {
    s_fail = 0;
    tc::mbar_init(&b_full, 1);
    for (int p = 0; p < kParts; ++p) {
      tc::mbar_init(&a_full[p], 1); tc::mbar_init(&a_empty[p], 1);
      tc::mbar_init(&tm_full[p], 1); tc::mbar_init(&tm_empty[p], kTcEpiWarps / kParts);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {                                           // 512 columns: one 128 x 128 fp32 accumulator per part
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
      const int n_box = (n_cols + kBBoxRows - 1) / kBBoxRows;    // rows past the slice's S are other slices' rows: never used
      tc::mbar_expect_tx(&b_full, (uint32_t)(KB * n_box * kBBoxRows * 128));
      for (int kb = 0; kb < KB; ++kb)
        for (int j = 0; j < n_box; ++j)
          tc::tma_load_2d(sB + kb * B_BLOCK + j * kBBoxRows * 128, &map_pool, kb * 64, (int)(row0 + c0 + j * kBBoxRows), &b_full);
      for (int i = 0; i < T; ++i) {                            // tile i goes to part i % 4, its k-th tile with k = i / 4
        const int p = i % kParts, k = i / kParts;
        if (k >= 1 && !s_fail && !tc::mbar_wait(&a_empty[p], (uint32_t)((k - 1) & 1))) s_fail = 1;
        tc::mbar_expect_tx(&a_full[p], (uint32_t)A_TILE);
        for (int kb = 0; kb < KB; ++kb)
          tc::tma_load_2d(sA + p * A_TILE + kb * A_BLOCK, &map_k, kb * 64, slice * a.P + (t0 + i) * kTileM, &a_full[p]);
      }
    }
  } else if (warp == 1) {
    // ======================================================================= MMA issuer
    // Jobs are issued part by part in turn, so that while one part's epilogue drains its accumulator the tensor
    // cores work for the other three.
    if (lane == 0) {
      if (!tc::mbar_wait(&b_full, 0)) s_fail = 1;
      const int rounds = (T + kParts - 1) / kParts;
      for (int k = 0; k < rounds; ++k)
        for (int j = 0; j < n_j; ++j)
          for (int p = 0; p < kParts; ++p) {
            if (k * kParts + p >= T) continue;
            if (j == 0 && !s_fail && !tc::mbar_wait(&a_full[p], (uint32_t)(k & 1))) s_fail = 1;
            const int cnt = k * n_j + j;                         // jobs issued to this part before this one
            // the part's epilogue must have drained its accumulator (the first use passes at once)
            if (!s_fail && !tc::mbar_wait(&tm_empty[p], (uint32_t)((cnt & 1) ^ 1))) s_fail = 1;
            tc::fence_after_sync();
            const uint32_t d_tmem = tmem_base + (uint32_t)(p * kJobN);
            const uint32_t idesc = make_idesc(FMT, kTileM, j == n_j - 1 ? (uint32_t)n_last : (uint32_t)kJobN);
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
              const uint64_t adesc = tc::smem_desc_sw128(tc::smem_u32(sA + p * A_TILE + kb * A_BLOCK));
              const uint64_t bdesc = tc::smem_desc_sw128(tc::smem_u32(sB + kb * B_BLOCK + j * kJobN * 128));
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)                     // 16 elements = 32 bytes along K per instruction
                tc::mma_f16(d_tmem, adesc + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk), idesc, (kb | kk) != 0 ? 1u : 0u);
            }
            tc::mma_commit(&tm_full[p]);
            if (j == n_j - 1) tc::mma_commit(&a_empty[p]);       // the tile's slot is free once its MMAs have read it
          }
    }
  } else {
    // ======================================================================= epilogue warps
    // Four warps per part, one per quarter of the tensor-memory lanes: a thread owns one row of its part's prompt
    // tile and scans all retained columns of it, job after job, so that the row's maximum never leaves its registers
    // (no exchange between warps, no barrier per tile).
    const int e = warp - 2;
    const int quarter = warp & 3;                            // tensor-memory lanes this warp may read: 32*quarter ..
    const int p = e >> 2;                                    // part
    const int row = quarter * 32 + lane;                     // row of the prompt tile owned by this thread
    for (int i = tid - 64; i < kChunkN; i += kTcEpiWarps * 32)
      s_rn[i] = i < n_cols ? a.rnorm[row0 + c0 + i] : 0.f;
    asm volatile("bar.sync 1, %0;" ::"n"(kTcEpiWarps * 32) : "memory");
    unsigned long long* out_keys = a.part_key + ((size_t)slice * a.n_chunks_max + nc) * a.P;
    const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(p * kJobN);
    uint32_t ra[32], rb[32];
    const int n_tp = p < T ? (T - p + kParts - 1) / kParts : 0;   // tiles of this part
    // every load of a job has landed in registers: hand the accumulator back to the MMA warp
    auto release = [&]() {
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&tm_empty[p]);
    };
#pragma unroll 1
    for (int k = 0; k < n_tp; ++k) {
      float best = -INFINITY; int best_col = 0x7fffffff;
#pragma unroll 1
      for (int j = 0; j < n_j; ++j) {
        const int cnt = k * n_j + j;
        if (!s_fail && !tc::mbar_wait(&tm_full[p], (uint32_t)(cnt & 1))) s_fail = 1;
        tc::fence_after_sync();
        const int cl = j * kJobN;                              // chunk-local column of the job's first block
        const int nb = (min(kJobN, n_cols - cl) + 31) / 32;    // 32-column blocks with retained rows: 1 .. 4
        // loads run one block ahead of the scan
        tc::tmem_ld32_issue(lane_base, ra);
        tc::tmem_ld_wait(ra);
        if (nb > 1) tc::tmem_ld32_issue(lane_base + 32u, rb); else release();
        scan_block(ra, s_rn, cl, n_cols, c0, best, best_col);
        if (nb > 1) {
          tc::tmem_ld_wait(rb);
          if (nb > 2) tc::tmem_ld32_issue(lane_base + 64u, ra); else release();
          scan_block(rb, s_rn, cl + 32, n_cols, c0, best, best_col);
        }
        if (nb > 2) {
          tc::tmem_ld_wait(ra);
          if (nb > 3) tc::tmem_ld32_issue(lane_base + 96u, rb); else release();
          scan_block(ra, s_rn, cl + 64, n_cols, c0, best, best_col);
        }
        if (nb > 3) {
          tc::tmem_ld_wait(rb);
          release();
          scan_block(rb, s_rn, cl + 96, n_cols, c0, best, best_col);
        }
      }
      // (ordered value, inverted slot): larger is better, ties go to the lower slot; -0 counts as +0
      if (best == 0.f) best = 0.f;
      const unsigned long long key = best > -INFINITY
          ? (((unsigned long long)float_ord(best) << 32) | (uint32_t)(0x7fffffff - best_col)) : 0ull;
      const int pos = (t0 + k * kParts + p) * kTileM + row;
      if (pos < Pb) out_keys[pos] = key;
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc::fence_after_sync();
    tc::tmem_dealloc(tmem_base, 512);
  }
  if (tid == 0 && s_fail) report_error(a.status, D2O_ERR_TIMEOUT, 0x51C00000u | (uint32_t)(slice & 0xfffff));
}

// mx_i = 1/|k_i| * max over the chunks of the partial maxima, nn_i = its slot, for the evicted positions.
struct NnReduceArgs {
  const int32_t* budgets; const int64_t* row_off;
  const int32_t* evict_idx;
  const unsigned long long* part_key;
  const float* rnorm;                       // pool-wide 1/|k_c|
  float* evict_mx; int32_t* evict_nn;
  uint32_t* status;
  const int32_t* plen;
  int L, layer, Hkv, P, n_chunks_max;
};

constexpr int kNnRows = 4;                  // evicted rows per row group and pass: their loads are issued together

template <typename T, int D>
__global__ void __launch_bounds__(256)
neighbour_reduce_kernel(NnReduceArgs a, const T* __restrict__ K, const T* __restrict__ kpool) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int LPR = D / EPV;
  constexpr int NGRP = 256 / LPR;
  const int slice = blockIdx.y;
  const int b = slice / a.Hkv, h = slice % a.Hkv;
  const int S = a.budgets[slice_entry(b, a.layer, h, a.L, a.Hkv)];
  const int Pb = a.plen[b];
  const int Le = Pb - S;
  const int grp = threadIdx.x / LPR, lig = threadIdx.x % LPR;
  const int i0 = blockIdx.x * (NGRP * kNnRows) + grp;       // this group's rows: i0 + r * NGRP
  if (i0 >= Le) return;
  const unsigned gmask = group_mask<LPR>();
  const int n_chunks = (S + kChunkN - 1) / kChunkN;
  // The three dependent loads of a row (its position, its key, its partial maxima) are issued for four rows at a
  // time; the partial maxima of a row are spread over the lanes of its group (chunk c is lane c mod LPR's).
  int pos[kNnRows];
#pragma unroll
  for (int r = 0; r < kNnRows; ++r) {
    const int i = i0 + r * NGRP;
    pos[r] = i < Le ? a.evict_idx[(size_t)slice * a.P + i] : -1;
    if (pos[r] >= 0 && !D2O_GUARD(pos[r] < Pb, a.status, 0xC4EC0008u)) pos[r] = -1;    // uniform for the row's lanes
  }
  uint4 raw[kNnRows];
  unsigned long long key[kNnRows];
#pragma unroll
  for (int r = 0; r < kNnRows; ++r) {
    raw[r] = make_uint4(0, 0, 0, 0);
    key[r] = 0ull;
    if (pos[r] >= 0) {
      raw[r] = ld_global_v4(K + ((size_t)slice * a.P + pos[r]) * D + lig * EPV);
      for (int c = lig; c < n_chunks; c += LPR) {
        const unsigned long long k2 = a.part_key[((size_t)slice * a.n_chunks_max + c) * a.P + pos[r]];
        key[r] = k2 > key[r] ? k2 : key[r];
      }
    }
  }
#pragma unroll
  for (int r = 0; r < kNnRows; ++r) {
    if (pos[r] < 0) continue;                                // uniform for the row's lanes
    float f[EPV];
    Elem<T>::unpack(raw[r], f);
    float ss = 0.f;
#pragma unroll
    for (int e = 0; e < EPV; ++e) ss = fmaf(f[e], f[e], ss);
    ss = group_sum<LPR>(ss, gmask);
    const float rn = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
    unsigned long long kk = key[r];
#pragma unroll
    for (int o = LPR / 2; o >= 1; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(gmask, kk, o);
      kk = other > kk ? other : kk;
    }
    int slot = 0x7fffffff - (int)(uint32_t)(kk & 0xffffffffu);
    float mx = ord_float((uint32_t)(kk >> 32)) * rn;
    const bool found = kk != 0ull && (unsigned)slot < (unsigned)S;
    if (!found) {
      // No chunk reported a maximum (no finite similarity in the row: non-finite keys).  The row is redone here in
      // fp32, all retained rows in slot order (the first maximum stays); without any finite similarity it gets maximum
      // -inf and neighbour 0 and is never merged.
      const int64_t row0 = a.row_off[slice_entry(b, a.layer, h, a.L, a.Hkv)];
      float best = -INFINITY; int bj = 0;
      for (int j = 0; j < S; ++j) {
        float g[EPV];
        Elem<T>::unpack(ld_global_v4(kpool + (row0 + j) * D + lig * EPV), g);
        float dot = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) dot = fmaf(f[e], g[e], dot);
        dot = group_sum<LPR>(dot, gmask);
        const float u = __fadd_rn(dot * rn * a.rnorm[row0 + j], 0.f);
        if (u > best) { best = u; bj = j; }
      }
      mx = best; slot = bj;
    }
    if (lig == 0) {
      const int i = i0 + r * NGRP;
      a.evict_mx[(size_t)slice * a.P + i] = mx;
      a.evict_nn[(size_t)slice * a.P + i] = slot;
    }
  }
}

// ------------------------------------------------------------------------------------ host side
// The driver's tensor-map encoder, looked up through the runtime so that the library has no link-time dependency
// on the driver (it must load, and reject calls with status codes, on machines without one).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

bool encode_rows_2d(CUtensorMap* map, int dtype, const void* base, uint64_t rows, int d, int box_rows) {
  EncodeTiledFn encode = encode_tiled_fn();
  if (!encode) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)d * 2};
  const cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1u, 1u};
  const CUtensorMapDataType dt = dtype == D2O_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  return encode(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Upper bound of the work items of one layer: one per (slice, chunk) plus the splits into tile ranges.
size_t sim_tc_max_items(const d2o_config* cfg, int max_budget) {
  const size_t chunks = ((size_t)max_budget + kChunkN - 1) / kChunkN;
  return (size_t)cfg->batch * cfg->n_kv_heads * chunks + 2048;
}

// The work lists of all layers, built on the host once the budgets are known: every (slice, chunk of retained rows)
// is cut into ranges of prompt tiles of about equal work (tiles x columns), so that one launch is several full waves
// of CTAs of the same length whatever the spread of the budgets; longest first.  `items` has room for
// n_layers * sim_tc_max_items() entries, `count[layer]` receives the entries of each layer.
void sim_tc_build_items(const d2o_ctx* c, int n_sms, int4* items, int32_t* count) {
  const d2o_config& g = c->cfg;
  const int B = g.batch, Hkv = g.n_kv_heads, L = g.n_layers;
  const size_t cap = sim_tc_max_items(&g, c->max_budget);
  struct Piece { int slice, chunk, tiles, cols; };
  Piece* pieces = (Piece*)malloc(sizeof(Piece) * (size_t)B * Hkv * ((c->max_budget + kChunkN - 1) / kChunkN + 1));
  for (int layer = 0; layer < L; ++layer) {
    int4* out = items + (size_t)layer * cap;
    size_t n_pieces = 0;
    double total = 0.0;
    for (int b = 0; b < B; ++b)
      for (int h = 0; h < Hkv; ++h) {
        const int S = c->h_budgets[((size_t)b * L + layer) * Hkv + h];
        const int P = c->h_plen[b];
        if (P - S <= 0) continue;
        const int n_chunks = (S + kChunkN - 1) / kChunkN, cc = chunk_columns(S);
        const int tiles = (P + kTileM - 1) / kTileM;
        for (int nc = 0; nc < n_chunks; ++nc) {
          const int cols = min(cc, S - nc * cc);
          if (cols <= 0) continue;
          pieces[n_pieces++] = {b * Hkv + h, nc, tiles, cols};
          total += (double)tiles * (cols + 64);                // + a per-tile cost that does not depend on the columns
        }
      }
    size_t n = 0;
    if (n_pieces > 0) {
      // aim at five waves of equal items, at least eight tiles each (a CTA first loads its chunk of retained rows and keeps four tiles in flight)
      const double target = total / ((double)n_sms * 5.0);
      std::vector<std::pair<double, int4>> list;
      for (size_t i = 0; i < n_pieces; ++i) {
        const Piece& p = pieces[i];
        const double work = (double)p.tiles * (p.cols + 64);
        int k = (int)(work / target + 0.5);
        k = max(1, min(k, max(1, p.tiles / 8)));
        if (list.size() + k + (n_pieces - i) > cap) k = 1;     // never more entries than the list holds
        for (int j = 0; j < k; ++j) {
          const int t0 = (int)((long long)p.tiles * j / k), t1 = (int)((long long)p.tiles * (j + 1) / k);
          if (t1 > t0) list.push_back({(double)(t1 - t0) * (p.cols + 64), make_int4(p.slice, p.chunk, t0, t1)});
        }
      }
      // longest first; ties keep the slice order
      std::stable_sort(list.begin(), list.end(),
                       [](const std::pair<double, int4>& x, const std::pair<double, int4>& y) { return x.first > y.first; });
      for (const auto& e : list) out[n++] = e.second;
    }
    count[layer] = (int32_t)n;
  }
  free(pieces);
}

size_t sim_tc_part_key_bytes(const d2o_config* cfg, int max_budget) {
  const size_t chunks = ((size_t)max_budget + kChunkN - 1) / kChunkN;
  return (size_t)cfg->batch * cfg->n_kv_heads * chunks * cfg->prompt_len * 8;
}

// Returns cudaErrorNotSupported if the tensor maps cannot be built.
cudaError_t launch_similarity_tc(const d2o_ctx* c, int layer, const void* K, int max_S, cudaStream_t st, int lane) {
  const d2o_config& g = c->cfg;
  const int B = g.batch, Hkv = g.n_kv_heads, P = g.prompt_len, D = g.d_head;
  const int n_slices = B * Hkv;
  char* S = c->state; char* X = c->scratch + (size_t)lane * c->slay.lane_stride;   // only the lane's arrays are used below
  CUtensorMap map_k, map_pool;
  if (!encode_rows_2d(&map_k, g.dtype, K, (uint64_t)n_slices * P, D, kTileM)) return cudaErrorNotSupported;
  // the retained rows of the same kind: K_c, or V_c when the similarity is taken on the values
  char* pool = S + (g.sim_feature ? c->lay.vpool : c->lay.kpool);
  if (!encode_rows_2d(&map_pool, g.dtype, pool, (uint64_t)c->pool_rows, D, kBBoxRows)) return cudaErrorNotSupported;
  const int n_chunks_max = (c->max_budget + kChunkN - 1) / kChunkN;
  (void)max_S;
  const int n_items = c->h_sim_count[layer];
  if (n_items == 0) return cudaSuccess;                      // nothing was evicted in this layer

  SimTcArgs a;
  a.budgets = (const int32_t*)(S + c->lay.budgets); a.row_off = (const int64_t*)(S + c->lay.row_off);
  a.rnorm = (const float*)(S + c->lay.rnorm);
  a.part_key = (unsigned long long*)(X + c->slay.part_key);
  a.status = (uint32_t*)(S + c->lay.status);
  a.plen = (const int32_t*)(S + c->lay.plen);
  a.L = g.n_layers; a.layer = layer; a.Hkv = Hkv; a.P = P; a.n_chunks_max = n_chunks_max;
  a.items = (const int4*)(S + c->lay.sim_items) + (size_t)layer * sim_tc_max_items(&g, c->max_budget);
  const int KB = D / 64;
  const size_t smem = (size_t)KB * kChunkN * 128 + (size_t)kParts * KB * kTileM * 128 + kChunkN * 4;
  dim3 grid((unsigned)n_items);
  const int fmt = g.dtype == D2O_F16 ? 0 : 1;
  cudaError_t e;
#define D2O_LAUNCH_TC(DD, FF)                                                                                     \
  do {                                                                                                            \
    e = cudaFuncSetAttribute(sim_tc_kernel<DD, FF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);      \
    if (e != cudaSuccess) return e;                                                                               \
    sim_tc_kernel<DD, FF><<<grid, kTcThreads, smem, st>>>(a, map_k, map_pool);                                    \
  } while (0)
  if (D == 128) { if (fmt == 0) D2O_LAUNCH_TC(128, 0); else D2O_LAUNCH_TC(128, 1); }
  else          { if (fmt == 0) D2O_LAUNCH_TC(64, 0); else D2O_LAUNCH_TC(64, 1); }
#undef D2O_LAUNCH_TC
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;

  NnReduceArgs r;
  r.budgets = a.budgets; r.row_off = a.row_off; r.rnorm = a.rnorm; r.status = a.status; r.plen = a.plen;
  r.evict_idx = (const int32_t*)(X + c->slay.evict_idx); r.part_key = a.part_key;
  r.evict_mx = (float*)(X + c->slay.evict_mx); r.evict_nn = (int32_t*)(X + c->slay.evict_nn);
  r.L = g.n_layers; r.layer = layer; r.Hkv = Hkv; r.P = P; r.n_chunks_max = n_chunks_max;
  int maxLe = 0;
  for (int bb = 0; bb < B; ++bb)
    for (int hh = 0; hh < Hkv; ++hh) maxLe = max(maxLe, c->h_plen[bb] - c->h_budgets[(bb * g.n_layers + layer) * Hkv + hh]);
  if (maxLe <= 0) return cudaSuccess;
  const int lpr = D * 2 / 16;
  const int rows_per_cta = (256 / lpr) * kNnRows;
  dim3 rgrid((maxLe + rows_per_cta - 1) / rows_per_cta, n_slices);
  if (g.dtype == D2O_F16) {
    if (D == 128) neighbour_reduce_kernel<__half, 128><<<rgrid, 256, 0, st>>>(r, (const __half*)K, (const __half*)pool);
    else neighbour_reduce_kernel<__half, 64><<<rgrid, 256, 0, st>>>(r, (const __half*)K, (const __half*)pool);
  } else {
    if (D == 128) neighbour_reduce_kernel<__nv_bfloat16, 128><<<rgrid, 256, 0, st>>>(r, (const __nv_bfloat16*)K, (const __nv_bfloat16*)pool);
    else neighbour_reduce_kernel<__nv_bfloat16, 64><<<rgrid, 256, 0, st>>>(r, (const __nv_bfloat16*)K, (const __nv_bfloat16*)pool);
  }
  return cudaGetLastError();
}

}  // namespace d2o
