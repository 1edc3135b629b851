// Token generation (Section 3, Eq. 2-3; Section 4.2, Eq. 6-12): one fused kernel per decode step.
//
// One CTA handles one slice = (layer, sequence, KV head) with its G query heads, and streams the
// slice's cache rows through a ring of shared-memory stages filled by bulk asynchronous copies
// (cp.async.bulk, completion on mbarriers).  A producer warp runs ahead of the consumer warps by
// the depth of the ring, across the boundary of the two passes, so the reductions between them
// do not drain the memory pipeline:
//
//   guess    before the keys arrive: the rows with the lowest accumulated scores among those that may
//            be evicted in this step (Eq. 7-8) are the likely victims; their keys join the queries
//   pass K   keys once from HBM: logits of the G heads and the dot products with the guessed victims
//            (Eq. 9), the new token's row from the inputs
//            -> softmax normaliser -> AttnScore += probabilities (Eq. 6 case 2)
//            -> victim = lowest score outside the T sinks and the M most recent positions (Eq. 7-8)
//            -> if it was guessed (it nearly always is), its cosines are already there; if not, the
//               keys are read once more, directly from L2, for this one slice
//            -> nearest neighbour, tau_t (Eq. 10), merge decision, merged key row (Eq. 11-12)
//   pass V   values once from HBM: outputs (Eq. 3); the value rows of the victim and of the
//            neighbour are picked out of the stream for the merge (Eq. 11)
//   then     merged value row, the new token takes the victim's row.
// The guess changes no result: the victim is always the exact arg-min of the updated scores, and the
// cosines of a guessed row are the same dot products a second pass would compute.
// Everything that needs the whole slice is a block-wide reduction inside one CTA; there is no
// inter-CTA communication.
//
// Arithmetic: fp32 FMAs on unpacked rows (one query head per KV head, or fp32 caches), or, for 16-bit caches with
// grouped queries, mma.sync for both passes on stages that arrive through tiled tensor maps with the 128-byte
// swizzle.  A decode step over all layers runs the slices largest first and, where a few slices are much longer
// than the rest, those in a launch of their own with sixteen consumer warps (see launch_decode).
#include <math.h>

#include <cuda/std/type_traits>

#include "d2o_common.cuh"
#include "d2o_tc.cuh"

namespace d2o {

// Consumer warps per CTA (CW) are a template parameter: 4 for many small slices (more CTAs per SM hide the
// reductions between the passes), 8 by default, 16 for few large slices with grouped queries (one CTA per SM that
// streams twice as fast).  A CTA has CW consumer warps + one producer warp; every consumer thread reads four 16-byte
// vectors per stage.
__host__ __device__ constexpr int stage_bytes_of(int cw) { return 4 * cw * 32 * 16; }
constexpr int kMaxStages = 12;
constexpr unsigned long long kWaitNs = 1000000000ull;   // an mbarrier wait gives up after 1 s
constexpr int kTensorMinG = 2;                          // query heads per KV head from which the tensor-core path is used
constexpr uint32_t kSuspendNs = 4000u;                  // a waiting thread may stay suspended this long before it looks again

struct DecodeArgs {
  const int32_t* budgets; const int32_t* windows; const int64_t* row_off;   // [B, L, Hkv]
  int32_t* pos; float* score; float* rnorm;                                  // pool-wide
  int32_t* len; float* tau;                                                  // [L, B, Hkv]
  unsigned long long* counters; uint32_t* status;
  const int32_t* plen;              // [B] prompt length of every sequence
  int L, l0, B, Hkv, T, step;       // step = number of tokens generated before this one: its position is plen[b] + step
  float beta, tau_override;
  int row_cap;                      // rows of a slice whose logits / probabilities live in shared memory (multiple of 8)
  float* spill;                     // the same for rows >= row_cap: [(row0 + 8 slice) G + g (stride(S) + 8) + row], stays in L2
  int stages;                       // stages of the ring
  int l2_hints;                     // 1: the streamed rows are marked evict-first in L2 (each is read once per step)
  const int32_t* order;             // NULL: CTAs take (layer, b, h) in index order; else (layer * B + b) per group of Hkv CTAs
  int pair_base;                    // first entry of `order` this launch works on
  int average;                      // 1: average merge (both rows weigh 1/2) instead of the weights of Eq. 12
  unsigned long long wait_ns;       // a wait for a stage gives up after this long
  int stop_stage;                   // failure-detection tests: the producer issues no copy from this stage on (-1: never)
  long long pool_rows;              // rows of the cache pool (bounds of the checked build)
  int32_t* steps_done;              // [L, B, Hkv] decode steps completed on the slice: written as a CTA's last act
  int chained;                      // 1: the previous step's grids may still be running (see slice_ready)
  int publish;                      // 1: a chained step follows: the CTA publishes the slice's step counter at its end
};

// ----------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long global_ns() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
template <int CW>
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(CW * 32) : "memory"); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(kSuspendNs) : "memory");
  return ok != 0;
}
// Wait for a stage in the kernel's loops: one probe when the phase is already complete (the common case); otherwise
// poll until it completes, another thread has recorded a timeout, or this one does.
__device__ __forceinline__ void stage_wait(unsigned long long* bar, uint32_t parity, volatile int* timeout,
                                           unsigned long long limit_ns) {
  if (mbar_try_wait(bar, parity)) return;
  const unsigned long long t0 = global_ns();
  while (*timeout == 0) {
    if (mbar_try_wait(bar, parity)) return;
    if (global_ns() - t0 > limit_ns) { *timeout = 2; return; }
  }
}
// The same without giving up early when another thread has recorded a timeout: used by the producer to see its own
// copies land before it leaves.  false = the limit ran out.
__device__ __forceinline__ bool landed_wait(unsigned long long* bar, uint32_t parity, unsigned long long limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  while (!mbar_try_wait(bar, parity))
    if (global_ns() - t0 > limit_ns) return false;
  return true;
}
// Waits, with a limit, until the slice's step counter has reached `want`: the CTA that ran the slice's previous
// decode step has finished and its stores are visible.  0: ready; 1: an anomaly was recorded meanwhile (the state is
// no longer trusted); 2: the wait ran out.
__device__ __forceinline__ int slice_ready(const int32_t* flag, int want, const uint32_t* status, unsigned long long limit_ns) {
  const unsigned long long t0 = global_ns();
  for (;;) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
    if (v >= want) return 0;
    if (*reinterpret_cast<const volatile uint32_t*>(status) != 0u) return 1;
    if (global_ns() - t0 > limit_ns) return 2;
    __nanosleep(200);
  }
}
// Similarity as an ordered key: -0 (a zero-norm row times a negative dot product) must count as +0, or equal
// similarities would not tie.
__device__ __forceinline__ uint32_t sim_ord(float u) { return float_ord(__fadd_rn(u, 0.f)); }
// d = a * b + c on two fp32 lanes at once (one issue slot instead of two)
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;"
      : "=l"(d)
      : "l"(*reinterpret_cast<const unsigned long long*>(&a)), "l"(*reinterpret_cast<const unsigned long long*>(&b)),
        "l"(*reinterpret_cast<const unsigned long long*>(&c)));
  return *reinterpret_cast<float2*>(&d);
}
// dot product of two pieces of N floats each, accumulated in two interleaved fp32 chains
template <int N>
__device__ __forceinline__ float dot_pairs(const float (&a)[N], const float (&b)[N]) {
  float2 acc = make_float2(0.f, 0.f);
#pragma unroll
  for (int i = 0; i < N; i += 2) acc = ffma2(make_float2(a[i], a[i + 1]), make_float2(b[i], b[i + 1]), acc);
  return acc.x + acc.y;
}
// next slot of the ring; the parity flips on wrap-around
__device__ __forceinline__ void ring_next(int& slot, uint32_t& ph, int stages) {
  if (++slot == stages) { slot = 0; ph ^= 1u; }
}
// global -> this CTA's shared memory, 16-byte aligned on both sides, size a multiple of 16
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_g2s_hint(void* dst, const void* src, uint32_t bytes, unsigned long long* bar,
                                              unsigned long long policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy) : "memory");
}

// 2-D tiled load with an L2 eviction-priority hint; x = innermost coordinate (elements), y = row
__device__ __forceinline__ void tma_load_2d_hint(void* dst, const CUtensorMap* map, int x, int y, unsigned long long* bar,
                                                 unsigned long long policy) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
               ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy) : "memory");
}

// Extremum over the consumer warps of a 64-bit key with the row index of the winner (keys are unique per row).
// The result is valid in s_out_key / s_out_li after the next consumer_sync().
template <bool MIN, int CW>
__device__ __forceinline__ void block_arg_extreme(unsigned long long key, int li, unsigned long long* s_key,
                                                   int* s_li, unsigned long long* s_out_key, int* s_out_li) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned long long w = MIN ? warp_min_u64(key) : warp_max_u64(key);
  const unsigned vote = __ballot_sync(0xffffffffu, key == w);
  const int src = __ffs(vote) - 1;
  const int wli = __shfl_sync(0xffffffffu, li, src);
  if (lane == 0) { s_key[warp] = w; s_li[warp] = wli; }
  consumer_sync<CW>();
  if (threadIdx.x == 0) {
    unsigned long long b = s_key[0]; int bl = s_li[0];
    for (int i = 1; i < CW; ++i) {
      const bool better = MIN ? (s_key[i] < b) : (s_key[i] > b);
      if (better) { b = s_key[i]; bl = s_li[i]; }
    }
    *s_out_key = b; *s_out_li = bl;
  }
}

// Sums four values, each spread over the LPR lanes of a row group, with 3 + log2(LPR/4) shuffles instead of
// 4*log2(LPR): lanes trade halves of the batch first.  Lane `lig` returns the total of value lig / (LPR/4).
// All 32 lanes of the warp must call it.
template <int LPR>
__device__ __forceinline__ float reduce4(float s0, float s1, float s2, float s3, int lig) {
  const bool hi = (lig & (LPR / 2)) != 0;
  float k0 = hi ? s2 : s0, k1 = hi ? s3 : s1;
  const float t0 = hi ? s0 : s2, t1 = hi ? s1 : s3;
  k0 += __shfl_xor_sync(0xffffffffu, t0, LPR / 2);
  k1 += __shfl_xor_sync(0xffffffffu, t1, LPR / 2);
  const bool hi2 = (lig & (LPR / 4)) != 0;
  float k = hi2 ? k1 : k0;
  const float t = hi2 ? k0 : k1;
  k += __shfl_xor_sync(0xffffffffu, t, LPR / 4);
#pragma unroll
  for (int o = LPR / 8; o > 0; o >>= 1) k += __shfl_xor_sync(0xffffffffu, k, o);
  return k;
}

// One warp-level tensor-core step for the logits of 16 rows against up to 8 heads: acc (16 x 8, fp32) += A (16 rows x
// 16 elements of d, from the row-major stage) * B (16 elements x 8 heads, the queries).  Both operands take their
// 16-byte pieces from the same offsets of their rows, so the order of the elements inside a step is free and a
// thread's piece is one contiguous vector load.
// the same step with a zero accumulator on input: d = a * b
template <typename T>
__device__ __forceinline__ void mma_16x8x16_zero(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                 uint32_t b0, uint32_t b1) {
  if constexpr (sizeof(T) == 2 && !cuda::std::is_same<T, __nv_bfloat16>::value) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
  } else {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
  }
}
template <typename T>
__device__ __forceinline__ void mma_16x8x16(float (&acc)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                            uint32_t b0, uint32_t b1) {
  if constexpr (sizeof(T) == 2 && !cuda::std::is_same<T, __nv_bfloat16>::value) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(acc[0]), "+f"(acc[1]), "+f"(acc[2]), "+f"(acc[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  } else {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(acc[0]), "+f"(acc[1]), "+f"(acc[2]), "+f"(acc[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
}

// (hi, lo) 16-bit pairs of two fp32 weights, hi + lo carrying 16 (bf16) or 22 (fp16) significant bits: x -> low half
template <typename T>
__device__ __forceinline__ void split_pair(float x, float y, uint32_t& hi, uint32_t& lo) {
  if constexpr (cuda::std::is_same<T, __nv_bfloat16>::value) {
    // hi = the upper 16 bits (the subtraction is then exact), lo = the remainder rounded
    const uint32_t xb = __float_as_uint(x) & 0xffff0000u, yb = __float_as_uint(y) & 0xffff0000u;
    hi = (xb >> 16) | yb;
    const __nv_bfloat162 l = __floats2bfloat162_rn(x - __uint_as_float(xb), y - __uint_as_float(yb));
    lo = *reinterpret_cast<const uint32_t*>(&l);
  } else {
    const __half xh = __float2half_rn(x), yh = __float2half_rn(y);
    const __half2 h = __halves2half2(xh, yh);
    const __half2 l = __halves2half2(__float2half_rn(x - __half2float(xh)), __float2half_rn(y - __half2float(yh)));
    hi = *reinterpret_cast<const uint32_t*>(&h); lo = *reinterpret_cast<const uint32_t*>(&l);
  }
}
// four 8x8 16-bit matrices, transposed on the way into registers (value rows become the A operand's columns)
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t saddr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(saddr) : "memory");
}

// Dot products of the 16 rows of tile `tile` of a swizzled stage ([d half][SR rows][128 bytes], 16-byte chunk c of
// row r at chunk c ^ (r & 7)) with the (up to 8) vectors whose fragments are in `qb`.  Thread (gid, tig) reads chunk
// 2 tig + (j & 1) of half j / 2 of rows gid and gid + 8 in step j: with the swizzle the eight lanes of a quarter-warp
// hit eight different bank groups.  The order of the elements inside a step is free as long as both operands agree,
// so a thread's piece is one vector load; `qb[j]` holds the same chunk of vector gid.
// acc[0], acc[1] = row gid of the tile against vectors 2 tig, 2 tig + 1; acc[2], acc[3] = row gid + 8.
template <typename T, int D, int SR>
__device__ __forceinline__ void tile_dots(const unsigned char* stage, int tile, const uint4 (&qb)[D / 32], float (&acc)[4]) {
  const int gid = (threadIdx.x & 31) >> 2, tig = threadIdx.x & 3;
  // all fragments first, then one tensor-core step per 16 elements of d, each into its own accumulator: neither
  // the loads nor the steps wait for one another
  uint4 A0[D / 32], A1[D / 32];
#pragma unroll
  for (int j = 0; j < D / 32; ++j) {
    const unsigned char* row = stage + (size_t)(j >> 1) * SR * 128 + (size_t)(tile * 16 + gid) * 128 +
                               (((2 * tig + (j & 1)) ^ gid) << 4);
    A0[j] = *reinterpret_cast<const uint4*>(row);
    A1[j] = *reinterpret_cast<const uint4*>(row + 8 * 128);
  }
  float part[D / 16][4];
#pragma unroll
  for (int j = 0; j < D / 32; ++j) {
    mma_16x8x16_zero<T>(part[2 * j], A0[j].x, A1[j].x, A0[j].y, A1[j].y, qb[j].x, qb[j].y);
    mma_16x8x16_zero<T>(part[2 * j + 1], A0[j].z, A1[j].z, A0[j].w, A1[j].w, qb[j].z, qb[j].w);
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < D / 16; ++i) t += part[i][e];
    acc[e] = t;
  }
}

// 16-bit caches take the tensor-core path (more registers per thread, fewer instructions per row)
__host__ __device__ constexpr bool tensor_path(int elem_size, int G) { return elem_size == 2 && G >= kTensorMinG; }
// CTAs per SM the kernel is compiled for
__host__ __device__ constexpr int ctas_per_sm(int cw, int G, int elem_size) {
  const bool t = tensor_path(elem_size, G);
  return cw == 4 ? (G <= 2 ? (t ? 5 : 7) : 4) : (cw == 8 ? (G <= 2 ? (t ? 3 : 4) : 2) : (G <= 2 && !t ? 2 : 1));
}

// OCC = CTAs per SM the registers are capped for (0: the table above)
template <typename T, int D, int G, int CW, int OCC = 0>
__global__ void __launch_bounds__((CW + 1) * 32, OCC > 0 ? OCC : ctas_per_sm(CW, G, (int)sizeof(T)))
decode_kernel(DecodeArgs a, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
              const T* __restrict__ q_in,
              const T* __restrict__ k_in, const T* __restrict__ v_in, T* __restrict__ out, T* __restrict__ kpool,
              T* __restrict__ vpool) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int LPR = D / EPV;                  // lanes that share one row (16-byte segment each)
  constexpr int kConsWarps = CW, kConsThreads = CW * 32, kStageBytes = stage_bytes_of(CW);
  constexpr int NGRP = kConsThreads / LPR;      // row groups of the consumers
  constexpr int SR = 4 * NGRP;                  // rows per stage: four per consumer thread
  constexpr int QL = LPR / 4;                   // lanes that end up with the same row total after reduce4
  constexpr int ROWB = D * (int)sizeof(T);      // bytes per row

  // 16-bit rows and several heads per KV head: logits, cosines and outputs on mma.sync (with one head the FMA loops
  // are as fast and use every warp).  The value stages then arrive through a tiled tensor map with the 128-byte
  // swizzle, because the value pass reads them with transposing matrix loads, which would conflict eight ways on
  // row-major 256-byte rows.
  constexpr bool kTensor = tensor_path((int)sizeof(T), G);
  constexpr int kTiles = SR / 16;                                      // 16-row tiles per stage (tensor path)
  constexpr bool kHalfTiles = 2 * kTiles == CW;                        // half as many tiles as warps (256-byte rows)
  static_assert(!kTensor || kTiles == CW || kHalfTiles, "tile assignment of the tensor path");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // a launch that follows with programmatic stream serialisation (the short slices of the same step, which share
  // nothing with this one) may start as soon as every CTA of this one is running; its producer warps wait for this
  // grid to finish before they exit (griddepcontrol.wait below)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // ---- which slice: in index order, or largest caches first through the order table
  const int h = (int)blockIdx.x % a.Hkv;
  int layer, b;
  if (a.order) {
    const int pair = a.order[a.pair_base + (int)blockIdx.x / a.Hkv];
    layer = pair / a.B; b = pair % a.B;
  } else {
    layer = a.l0 + (int)blockIdx.x / (a.B * a.Hkv);
    b = ((int)blockIdx.x / a.Hkv) % a.B;
  }
  const int sl = ((layer - a.l0) * a.B + b) * a.Hkv + h;     // slice index within the call's q/k/v/out
  const T* k_new = k_in + (size_t)sl * D;
  const T* v_new = v_in + (size_t)sl * D;

  // ---- slice parameters
  const int t_pos = a.plen[b] + a.step;                                // position of the token generated in this step
  const int S = a.budgets[slice_entry(b, layer, h, a.L, a.Hkv)];
  const int M = a.windows[slice_entry(b, layer, h, a.L, a.Hkv)];
  const int64_t row0 = a.row_off[slice_entry(b, layer, h, a.L, a.Hkv)];
  const int sidx = (layer * a.B + b) * a.Hkv + h;
  // a chained step runs beside the grids of the step before it: the slice is this CTA's once that step's CTA has
  // published it
  __shared__ int s_chain;
  if (a.chained) {
    if (tid == 0) s_chain = slice_ready(a.steps_done + sidx, a.step, a.status, a.wait_ns);
    __syncthreads();
    if (s_chain != 0) {                                              // uniform for the CTA, before any barrier or copy
      if (tid == 0 && s_chain == 2) report_error(a.status, D2O_ERR_TIMEOUT, 0xDEC20000u | (uint32_t)(sl & 0xffff));
      return;
    }
  }
  const int n_old = a.len[sidx];
  const float tau_old = a.tau[sidx];
  if (!D2O_GUARD(S >= 1 && n_old >= 0 && n_old <= S && row0 >= 0 && row0 + slice_stride(S) <= a.pool_rows, a.status,
                 0xC4EC0010u))
    return;                                                          // uniform for the CTA, before any barrier or copy
  const int n = n_old + 1;                                         // rows attended: cache + the new token
  const int Tn = a.T < S ? a.T : S;
  const bool evict = n > S;
  const int n_st = (n + SR - 1) / SR;                              // stages per pass
  const int NS = a.stages;

  // ---- shared memory
  extern __shared__ __align__(1024) unsigned char dsm[];
  uint4* ring = reinterpret_cast<uint4*>(dsm);                       // [stages][SR][LPR]
  float* red = reinterpret_cast<float*>(dsm);                        // [warps][G][D], aliases the ring once it is drained
  float* meta_rn = reinterpret_cast<float*>(dsm + (size_t)NS * kStageBytes);   // [stages][SR] 1/|k| of a pass-K' stage's rows
  int* meta_ps = reinterpret_cast<int*>(meta_rn + (size_t)NS * SR);  // [stages][SR] positions of a pass-K' stage's rows
  float* pl = reinterpret_cast<float*>(meta_ps + (size_t)NS * SR);   // [G][row_cap] logits -> probabilities
  uint4* stash = reinterpret_cast<uint4*>(pl + (size_t)G * a.row_cap);   // [2][LPR] value rows of the victim / the neighbour
  // rows beyond row_cap (slices much longer than most): same array in global memory, which the CTA rewrites every
  // step and which therefore stays in L2; 16 bytes per row against the 768 streamed for its key and value
  float* const pl_far = a.spill + (size_t)(row0 + 8 * (int64_t)sidx) * G;
  const int far_stride = slice_stride(S) + 8;
  auto pl_get = [&](int g, int li) -> float {
    if (li < a.row_cap) return pl[(size_t)g * a.row_cap + li];
    return pl_far[(size_t)g * far_stride + li];
  };
  auto pl_put = [&](int g, int li, float x) {
    if (li < a.row_cap) pl[(size_t)g * a.row_cap + li] = x;
    else pl_far[(size_t)g * far_stride + li] = x;
  };
  __shared__ unsigned long long s_full[kMaxStages], s_empty[kMaxStages];
  __shared__ float s_new_rn, s_new_score;                            // inverse key norm and accumulated score of the new token
  __shared__ float s_red[2][kConsWarps][G];
  __shared__ unsigned long long s_key[kConsWarps], s_best_key;
  __shared__ int s_li[kConsWarps], s_best_li;
  __shared__ volatile int s_timeout;                                 // 1: an earlier launch recorded an anomaly; 2: a wait of this CTA ran out
  __shared__ int s_bail;
  __shared__ unsigned long long s_done;                              // arrivals of the consumer warps at the kernel's end

  if (tid == 0) {
    s_timeout = *reinterpret_cast<volatile uint32_t*>(a.status) != 0u;
    for (int s = 0; s < NS; ++s) { mbar_init(&s_full[s], 1); mbar_init(&s_empty[s], kConsWarps); }
    mbar_init(&s_done, kConsWarps);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  // once an anomaly has been recorded the state is no longer trusted: later steps do nothing (the error word stays
  // set and the caller finds it with d2o_get_stats)
  if (s_timeout != 0) return;

  // =========================================================================== producer warp
  if (warp == kConsWarps) {
    if (lane == 0) {
      // rows that the previous step's CTA wrote with ordinary stores are read here by bulk copies
      if (a.chained) asm volatile("fence.proxy.async.global;" ::: "memory");
      unsigned long long drop = 0;
      if (a.l2_hints) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(drop));
      int slot = 0, q = 0;
      uint32_t ph = 1;                                               // parity of the previous use of a slot
      bool stopped = false;
      for (int p = 0; p < 2 && !stopped; ++p) {
        const bool is_v = (p == 1);
        const T* pool = is_v ? vpool : kpool;
        const T* fresh = is_v ? v_new : k_new;
        const bool hint = a.l2_hints != 0;
        // Keys and values cross once per step, so their lines are the first to leave L2; what stays is the per-row
        // state, which is read twice and written.  (Keeping the keys for the rare second look after a wrong guess
        // cost 3 - 8 % of the step; that look now goes to DRAM.)
        const unsigned long long pol = drop;
        for (int s = 0; s < n_st; ++s, ++q, ring_next(slot, ph, NS)) {
          if (q >= NS) stage_wait(&s_empty[slot], ph, &s_timeout, a.wait_ns);
          // a wait ran out somewhere in this CTA, or the failure-detection tests asked for a stage that never
          // arrives: nothing more is issued
          if (s_timeout != 0 || (a.stop_stage >= 0 && q >= a.stop_stage)) { stopped = true; break; }
          const int a0 = s * SR, a1 = min(n, a0 + SR);
          const int np = max(0, min(a1, n_old) - a0);                // cache rows of the stage
          const bool nw = n_old >= a0 && n_old < a1;                 // the new token's row falls into the stage
          uint4* dst = ring + (size_t)slot * SR * LPR;
          // the cosines of pass K also need 1/|k| and the position of the rows (16-byte granules: up to 3 entries past
          // n_old come from the slice's padding and are never used)
          const bool with_meta = evict && p == 0 && np > 0;
          const int np4 = (np + 3) & ~3;
          if (kTensor) {
            // swizzled [d half][SR rows][128 B]; the box always has SR rows (what lies past the cache rows is never
            // used, or zeroed by the consumers); the new token's rows are not in the stream: its logits, its cosine
            // and its term of the output are added from the inputs
            mbar_expect_tx(&s_full[slot], (uint32_t)(SR * ROWB + (with_meta ? 2 * np4 * 4 : 0)));
            if (with_meta) {
              bulk_g2s(meta_rn + (size_t)slot * SR, a.rnorm + row0 + a0, (uint32_t)(np4 * 4), &s_full[slot]);
              bulk_g2s(meta_ps + (size_t)slot * SR, a.pos + row0 + a0, (uint32_t)(np4 * 4), &s_full[slot]);
            }
            const CUtensorMap* map = is_v ? &map_v : &map_k;
#pragma unroll
            for (int hf = 0; hf < ROWB / 128; ++hf) {
              void* to = reinterpret_cast<unsigned char*>(dst) + (size_t)hf * SR * 128;
              if (hint) tma_load_2d_hint(to, map, hf * 64, (int)(row0 + a0), &s_full[slot], pol);
              else tc::tma_load_2d(to, map, hf * 64, (int)(row0 + a0), &s_full[slot]);
            }
            continue;
          }
          mbar_expect_tx(&s_full[slot], (uint32_t)((np + (nw ? 1 : 0)) * ROWB + (with_meta ? 2 * np4 * 4 : 0)));
          if (with_meta) {
            bulk_g2s(meta_rn + (size_t)slot * SR, a.rnorm + row0 + a0, (uint32_t)(np4 * 4), &s_full[slot]);
            bulk_g2s(meta_ps + (size_t)slot * SR, a.pos + row0 + a0, (uint32_t)(np4 * 4), &s_full[slot]);
          }
          if (np > 0) {
            if (hint) bulk_g2s_hint(dst, pool + (row0 + a0) * D, (uint32_t)(np * ROWB), &s_full[slot], pol);
            else bulk_g2s(dst, pool + (row0 + a0) * D, (uint32_t)(np * ROWB), &s_full[slot]);
          }
          if (nw) bulk_g2s(dst + (size_t)(n_old - a0) * LPR, fresh, (uint32_t)ROWB, &s_full[slot]);
        }
      }
      if (stopped) {
        // The consumers will run into a wait that gives up and may leave early.  The CTA must not end while copies
        // are on their way into its shared memory: see the last (up to NS) issued stages land, each wait bounded.
        const int n_back = q < NS ? q : NS;
        int sl_i = slot; uint32_t ph_i = ph;                         // `slot` is the stage that was not issued
        for (int i = 0; i < n_back; ++i) {
          if (sl_i == 0) { sl_i = NS - 1; ph_i ^= 1u; } else --sl_i;
          if (!landed_wait(&s_full[sl_i], ph_i ^ 1u, a.wait_ns)) break;
        }
      }
      // a chained step follows: once every consumer warp has arrived (the slice's state is complete and ordered
      // before this thread by the arrivals), publish the slice's step counter.  Not after a wait ran out: the step
      // after this one then finds the error word, or runs into its own limit.
      if (a.publish && !stopped) {
        stage_wait(&s_done, 0u, &s_timeout, a.wait_ns);
        if (s_timeout == 0)
          asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(a.steps_done + sidx), "r"(a.step + 1) : "memory");
      }
    }
    // A grid launched with programmatic stream serialisation may run beside its predecessor, but it must not be
    // complete before it: whatever the stream runs next (the next step, a copy of the outputs) is ordered behind
    // this grid only.  One CTA that stays until the predecessor has finished is enough for that, and keeps the other
    // CTAs' places free for the rest of this grid: the last one, which holds the shortest slice.  The instruction
    // returns at once in an ordinarily launched grid.
    if (blockIdx.x == gridDim.x - 1) asm volatile("griddepcontrol.wait;" ::: "memory");
    return;
  }

  // =========================================================================== consumer warps
  // the accumulated scores and positions of the rows are needed right after pass K: ask L2 for their lines now
  for (int i = tid * 32; i < n_old; i += kConsThreads * 32) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(a.score + row0 + i));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(a.pos + row0 + i));
  }
  const int grp = tid / LPR, lig = tid % LPR;
  const unsigned gmask = group_mask<LPR>();
  int slot = 0;                                                      // ring position and parity, running across the passes
  uint32_t ph = 0;

  const float qscale = (D == 64 ? 0.125f : 0.08838834764831845f) * kLog2e;   // log2(e)/sqrt(d)
  const int gid = lane >> 2, tig = lane & 3;
  // ---- query fragments: fp32, pre-scaled (FMA path) or raw 16-bit pieces of query `gid` (tensor path)
  float qf[kTensor ? 1 : G][EPV];
  uint4 qb[D / 32];
  if constexpr (kTensor) {
#pragma unroll
    for (int j = 0; j < D / 32; ++j)
      qb[j] = gid < G ? ld_global_v4(q_in + ((size_t)sl * G + gid) * D + ((j >> 1) * 8 + 2 * tig + (j & 1)) * 8)
                      : make_uint4(0, 0, 0, 0);
  } else {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float f[EPV];
      Elem<T>::unpack(ld_global_v4(q_in + ((size_t)sl * G + g) * D + lig * EPV), f);
#pragma unroll
      for (int e = 0; e < EPV; ++e) qf[g][e] = f[e] * qscale;
    }
  }
  // the new token's rows, kept by the first row group
  uint4 knew = make_uint4(0, 0, 0, 0), vnew = make_uint4(0, 0, 0, 0);
  if (grp == 0) { knew = ld_global_v4(k_new + lig * EPV); vnew = ld_global_v4(v_new + lig * EPV); }

  // ---- guess of the victim: the NC rows with the lowest accumulated score (ties: the later position) among the rows
  // that may be evicted in this step, taken from the scores as they stand before the step (Eq. 7-8 on the old scores).
  // This step's probabilities are small against the differences between accumulated scores, so the victim that is
  // chosen after the softmax is nearly always one of them.  Their keys are multiplied with every row during pass K.
  constexpr int NC = kTensor ? 2 : 1;
  constexpr int kCandTig = G < 8 ? G / 2 : 0;                          // tensor path: the lanes whose columns hold the candidates
  int cand_li[NC];                                                     // row of candidate c in the slice, -1: none
  float cand_rn[NC];                                                   // its 1/|k|
  unsigned long long cbest[NC];                                        // this thread's best (cosine, earliest position) per candidate
  int cbest_li[NC];
  float ck[kTensor ? 1 : NC][EPV];                                     // FMA path: this lane's piece of the candidates' keys
  uint4 cb[D / 32];                                                    // tensor path, G = 8: fragments of candidate `gid`
#pragma unroll
  for (int c = 0; c < NC; ++c) { cand_li[c] = -1; cand_rn[c] = 0.f; cbest[c] = 0ull; cbest_li[c] = -1; }
#pragma unroll
  for (int j = 0; j < D / 32; ++j) cb[j] = make_uint4(0, 0, 0, 0);
  if (evict) {
    if (warp == 0) {
      // the new token's inverse norm, from the row as stored
      float f[EPV];
      Elem<T>::unpack(knew, f);
      float ss = 0.f;
#pragma unroll
      for (int e = 0; e < EPV; ++e) ss = fmaf(f[e], f[e], ss);
      ss = warp_sum(ss);                                               // lanes >= LPR hold zeros
      if (lane == 0) s_new_rn = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
    }
    unsigned long long my[NC];
    int my_li[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) { my[c] = ~0ull; my_li[c] = -1; }
    auto offer = [&](float sc, int pz, int li) {
      if (pz >= Tn && pz <= t_pos - M) {
        unsigned long long key = ((unsigned long long)float_ord(sc) << 32) | (uint32_t)(0x7fffffff - pz);
        int kl = li;
#pragma unroll
        for (int c = 0; c < NC; ++c)
          if (key < my[c]) { const unsigned long long tk = my[c]; const int tl = my_li[c]; my[c] = key; my_li[c] = kl; key = tk; kl = tl; }
      }
    };
    const int n_vec4 = (n_old / 4) * 4;
    for (int li = tid * 4; li < n_vec4; li += kConsThreads * 4) {
      const float4 sc = *reinterpret_cast<const float4*>(a.score + row0 + li);
      const int4 pz = *reinterpret_cast<const int4*>(a.pos + row0 + li);
      offer(sc.x, pz.x, li); offer(sc.y, pz.y, li + 1); offer(sc.z, pz.z, li + 2); offer(sc.w, pz.w, li + 3);
    }
    for (int li = n_vec4 + tid; li < n_old; li += kConsThreads) offer(a.score[row0 + li], a.pos[row0 + li], li);
    int taken = 0;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      unsigned long long k = ~0ull; int kl = -1;
#pragma unroll
      for (int j = 0; j < NC; ++j) if (taken == j) { k = my[j]; kl = my_li[j]; }
      block_arg_extreme<true, CW>(k, kl, s_key, s_li, &s_best_key, &s_best_li);
      consumer_sync<CW>();
      const unsigned long long bk = s_best_key;
      cand_li[c] = bk == ~0ull ? -1 : s_best_li;
      if (bk != ~0ull && bk == k) ++taken;                             // this thread's row was taken
    }
  }
  if (evict) {
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      if (cand_li[c] < 0) continue;
      const T* row = kpool + (row0 + cand_li[c]) * D;
      cand_rn[c] = a.rnorm[row0 + cand_li[c]];
      if constexpr (!kTensor) {
        Elem<T>::unpack(ld_global_v4(row + lig * EPV), ck[c]);
      } else if constexpr (G < 8) {
        // the candidates take the columns after the query heads of the same tensor-core steps
        if (gid == G + c) {
#pragma unroll
          for (int j = 0; j < D / 32; ++j) qb[j] = ld_global_v4(row + ((j >> 1) * 8 + 2 * tig + (j & 1)) * 8);
        }
      } else {
        if (gid == c) {
#pragma unroll
          for (int j = 0; j < D / 32; ++j) cb[j] = ld_global_v4(row + ((j >> 1) * 8 + 2 * tig + (j & 1)) * 8);
        }
      }
    }
    if constexpr (!kTensor) {
#pragma unroll
      for (int c = 0; c < NC; ++c)
        if (cand_li[c] < 0) {
#pragma unroll
          for (int e = 0; e < EPV; ++e) ck[c][e] = 0.f;
        }
    }
  }
  // cosine of row li (inverse norm rn, position pz) with candidate c, from their dot product: keeps this thread's best
  auto cand_update = [&](int c, float dot, float rn, int pz, int li) {
    if (li != cand_li[c]) {
      const unsigned long long key = ((unsigned long long)sim_ord(dot * cand_rn[c] * rn) << 32) | (uint32_t)(0x7fffffff - pz);
      if (key > cbest[c]) { cbest[c] = key; cbest_li[c] = li; }
    }
  };

  // ---- pass K: logits, and the candidates' dot products
  float mloc[G];
#pragma unroll
  for (int g = 0; g < G; ++g) mloc[g] = -INFINITY;
  const int n_plain_fma = min(n, a.row_cap);                        // FMA path: rows (the new token's included) with logits in shared memory
  if constexpr (kTensor) {
    // a stage has SR / 16 tiles of 16 rows.  With 256-byte rows that is half as many as there are warps: the lower
    // half of the warps takes the even stages, the upper half the odd ones (the others only hand the stage back), so
    // that two stages are worked on at a time.  With 128-byte rows every warp has a tile in every stage.  Thread
    // (gid, tig) ends up with rows gid, gid + 8 of its tile against heads 2 tig, 2 tig + 1
    float mm0 = -INFINITY, mm1 = -INFINITY;
    const int n_plain = min(n_old, a.row_cap);                       // rows whose logits go to shared memory unchecked
    // this warp's tile in the even / the odd stages (-1: none), and where its logits go
    const int tile_even = warp < kTiles ? warp : -1;
    const int tile_odd = kHalfTiles ? (warp >= kTiles ? warp - kTiles : -1) : warp;
    float* const pl_mine = pl + (size_t)(2 * tig) * a.row_cap + gid;
    for (int s = 0; s < n_st; ++s, ring_next(slot, ph, NS)) {
      stage_wait(&s_full[slot], ph, &s_timeout, a.wait_ns);
      const unsigned char* st = reinterpret_cast<const unsigned char*>(ring) + (size_t)slot * kStageBytes;
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      const int tile = (s & 1) ? tile_odd : tile_even;
      const int lt = s * SR + tile * 16;                             // first row of the tile
      const bool mine = tile >= 0 && lt < n_old;
      if (mine) tile_dots<T, D, SR>(st, tile, qb, acc);
      float acc2[4] = {0.f, 0.f, 0.f, 0.f};
      if constexpr (G == 8) {
        if (mine && evict) tile_dots<T, D, SR>(st, tile, cb, acc2);  // eight heads leave no column free: a second set of steps
      }
      // the candidates' columns belong to the lanes with tig = kCandTig: rows gid, gid + 8 of the tile; their 1/|k| and
      // positions leave the stage before it is released
      const bool cand_lane = evict && mine && tig == kCandTig;
      const int lr0 = tile * 16 + gid;
      float rn0 = 0.f, rn1 = 0.f; int ps0 = 0, ps1 = 0;
      if (cand_lane) {
        rn0 = meta_rn[(size_t)slot * SR + lr0]; ps0 = meta_ps[(size_t)slot * SR + lr0];
        rn1 = meta_rn[(size_t)slot * SR + lr0 + 8]; ps1 = meta_ps[(size_t)slot * SR + lr0 + 8];
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_empty[slot]);
      if (cand_lane) {
        const float* ca = G < 8 ? acc : acc2;
        if (lt + gid < n_old) { cand_update(0, ca[0], rn0, ps0, lt + gid); cand_update(1, ca[1], rn0, ps0, lt + gid); }
        if (lt + gid + 8 < n_old) { cand_update(0, ca[2], rn1, ps1, lt + gid + 8); cand_update(1, ca[3], rn1, ps1, lt + gid + 8); }
      }
      if (mine && 2 * tig < G) {
        const int li0 = lt + gid, li1 = li0 + 8;
        const float x00 = acc[0] * qscale, x01 = acc[1] * qscale, x10 = acc[2] * qscale, x11 = acc[3] * qscale;
        if (lt + 16 <= n_plain) {
          float* p = pl_mine + lt;
          p[0] = x00; p[8] = x10;
          mm0 = fmaxf(mm0, fmaxf(x00, x10));
          if (G > 1) {
            p[a.row_cap] = x01; p[a.row_cap + 8] = x11;
            mm1 = fmaxf(mm1, fmaxf(x01, x11));
          }
          continue;
        }
        if (li0 < n_old) {
          pl_put(2 * tig, li0, x00); mm0 = fmaxf(mm0, x00);
          if (2 * tig + 1 < G) { pl_put(2 * tig + 1, li0, x01); mm1 = fmaxf(mm1, x01); }
        }
        if (li1 < n_old) {
          pl_put(2 * tig, li1, x10); mm0 = fmaxf(mm0, x10);
          if (2 * tig + 1 < G) { pl_put(2 * tig + 1, li1, x11); mm1 = fmaxf(mm1, x11); }
        }
      }
    }
    // maxima over the rows (lanes with the same tig), then every lane gets every head's maximum
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
      mm0 = fmaxf(mm0, __shfl_xor_sync(0xffffffffu, mm0, o));
      mm1 = fmaxf(mm1, __shfl_xor_sync(0xffffffffu, mm1, o));
    }
#pragma unroll
    for (int g = 0; g < G; ++g) mloc[g] = __shfl_sync(0xffffffffu, (g & 1) ? mm1 : mm0, g >> 1);
    if (warp == 0) {
      // the new token's logits: its key row is held by the first LPR lanes
      float kf[EPV];
      Elem<T>::unpack(knew, kf);
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float qv[EPV];
        Elem<T>::unpack(lane < LPR ? ld_global_v4(q_in + ((size_t)sl * G + g) * D + lane * EPV) : make_uint4(0, 0, 0, 0), qv);
        float x = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) x = fmaf(qv[e], kf[e], x);
        x = warp_sum(x) * qscale;
        if (lane == 0) pl_put(g, n_old, x);
        mloc[g] = fmaxf(mloc[g], x);
      }
      if (evict) {
        // the new token is not in the stream: its cosines with the candidates come from the inputs
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          if (cand_li[c] < 0) continue;
          float cf[EPV];
          Elem<T>::unpack(lane < LPR ? ld_global_v4(kpool + (row0 + cand_li[c]) * D + lane * EPV) : make_uint4(0, 0, 0, 0), cf);
          float x = 0.f;
#pragma unroll
          for (int e = 0; e < EPV; ++e) x = fmaf(cf[e], kf[e], x);
          x = warp_sum(x);
          if (lane == 0) cand_update(c, x, s_new_rn, t_pos, n_old);
        }
      }
    }
  } else {
    for (int s = 0; s < n_st; ++s, ring_next(slot, ph, NS)) {
      stage_wait(&s_full[slot], ph, &s_timeout, a.wait_ns);
      const uint4* st = ring + (size_t)slot * SR * LPR + (size_t)grp * LPR + lig;   // this thread's piece of row grp
      const bool full = (s + 1) * SR <= n_plain_fma;                 // every row of the stage is a plain row
      uint4 raw[4];
      if (full) {
#pragma unroll
        for (int u = 0; u < 4; ++u) raw[u] = st[(size_t)u * NGRP * LPR];
      } else {
#pragma unroll
        for (int u = 0; u < 4; ++u)
          raw[u] = s * SR + u * NGRP + grp < n ? st[(size_t)u * NGRP * LPR] : make_uint4(0, 0, 0, 0);
      }
      float dot[G][4], cdot[NC][4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        float f[EPV];
        Elem<T>::unpack(raw[u], f);
#pragma unroll
        for (int g = 0; g < G; ++g) {
          dot[g][u] = dot_pairs<EPV>(qf[g], f);
        }
        if (evict) {
#pragma unroll
          for (int c = 0; c < NC; ++c) {
            cdot[c][u] = dot_pairs<EPV>(ck[c], f);
          }
        }
      }
      const int li = s * SR + (lig / QL) * NGRP + grp;               // the row whose total this lane receives
      // its 1/|k| and position leave the stage before the stage is released
      const bool cand_lane = evict && li < n && lig % QL == 0;
      float rn_li = s_new_rn; int ps_li = t_pos;
      if (cand_lane && li < n_old) { rn_li = meta_rn[(size_t)slot * SR + (li - s * SR)]; ps_li = meta_ps[(size_t)slot * SR + (li - s * SR)]; }
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_empty[slot]);
      if (evict) {
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          const float r = reduce4<LPR>(cdot[c][0], cdot[c][1], cdot[c][2], cdot[c][3], lig);
          if (cand_lane) cand_update(c, r, rn_li, ps_li, li);
        }
      }
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float r = reduce4<LPR>(dot[g][0], dot[g][1], dot[g][2], dot[g][3], lig);
        if (full) {
          mloc[g] = fmaxf(mloc[g], r);
          if (lig % QL == 0) pl[(size_t)g * a.row_cap + li] = r;
        } else if (li < n) {
          mloc[g] = fmaxf(mloc[g], r);
          if (lig % QL == 0) pl_put(g, li, r);
        }
      }
    }
  }
  // ---- softmax normaliser, probabilities, accumulated attention (Eq. 6 case 2), victim candidate
  if (warp == 0 && !evict) {
    // the new token's inverse norm from the row as stored (when a row is evicted it was needed before pass K)
    float f[EPV];
    Elem<T>::unpack(knew, f);
    float ss = 0.f;
#pragma unroll
    for (int e = 0; e < EPV; ++e) ss = fmaf(f[e], f[e], ss);
    ss = warp_sum(ss);                                               // lanes >= LPR hold zeros
    if (lane == 0) s_new_rn = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
  }
  float m_all[G], inv_l[G];
  {
#pragma unroll
    for (int g = 0; g < G; ++g) { const float w = warp_max(mloc[g]); if (lane == 0) s_red[0][warp][g] = w; }
    if (tid == 0) s_bail = s_timeout;
    consumer_sync<CW>();                                                 // logits, maxima and the new token's metadata
    if (s_bail != 0) {
      // a wait of the key pass ran out: the logits are not to be trusted, so nothing of the slice's state is touched
      if (tid == 0) report_error(a.status, D2O_ERR_TIMEOUT, 0xDEC10000u | (uint32_t)(sl & 0xffff));
      return;
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float t = s_red[0][0][g];
#pragma unroll
      for (int w = 1; w < kConsWarps; ++w) t = fmaxf(t, s_red[0][w][g]);
      m_all[g] = t;
    }
    float sum[G];
#pragma unroll
    for (int g = 0; g < G; ++g) sum[g] = 0.f;
    // cache rows with their logits in shared memory go four at a time; the last few, the new token and the rows
    // whose logits are in global memory one by one
    const int n_vec = (min(n_old, a.row_cap) / 4) * 4;
    for (int li = tid * 4; li < n_vec; li += kConsThreads * 4) {
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float4* p4 = reinterpret_cast<float4*>(pl + (size_t)g * a.row_cap + li);
        float4 x = *p4;
        x.x = exp2f(x.x - m_all[g]); x.y = exp2f(x.y - m_all[g]); x.z = exp2f(x.z - m_all[g]); x.w = exp2f(x.w - m_all[g]);
        *p4 = x;
        sum[g] += (x.x + x.y) + (x.z + x.w);
      }
    }
    for (int li = n_vec + tid; li < n; li += kConsThreads) {
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float p = exp2f(pl_get(g, li) - m_all[g]);
        pl_put(g, li, p);
        sum[g] += p;
      }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) { const float w = warp_sum(sum[g]); if (lane == 0) s_red[1][warp][g] = w; }
    consumer_sync<CW>();
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < kConsWarps; ++w) t += s_red[1][w][g];
      inv_l[g] = 1.0f / t;
    }
    unsigned long long my_min = ~0ull; int my_min_li = -1;
    for (int li = tid * 4; li < n_vec; li += kConsThreads * 4) {
      float4 p = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float4 x = *reinterpret_cast<const float4*>(pl + (size_t)g * a.row_cap + li);
        p.x = fmaf(x.x, inv_l[g], p.x); p.y = fmaf(x.y, inv_l[g], p.y);
        p.z = fmaf(x.z, inv_l[g], p.z); p.w = fmaf(x.w, inv_l[g], p.w);
      }
      float4* sc = reinterpret_cast<float4*>(a.score + row0 + li);
      float4 sn = *sc;
      sn.x += p.x; sn.y += p.y; sn.z += p.z; sn.w += p.w;
      *sc = sn;
      if (evict) {                                                   // lowest score, ties -> latest position
        const int4 pz = *reinterpret_cast<const int4*>(a.pos + row0 + li);
        const float sv[4] = {sn.x, sn.y, sn.z, sn.w};
        const int pv[4] = {pz.x, pz.y, pz.z, pz.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (pv[j] >= Tn && pv[j] <= t_pos - M) {
            const unsigned long long key = ((unsigned long long)float_ord(sv[j]) << 32) | (uint32_t)(0x7fffffff - pv[j]);
            if (key < my_min) { my_min = key; my_min_li = li + j; }
          }
        }
      }
    }
    for (int li = n_vec + tid; li < n; li += kConsThreads) {
      float p = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g) p = fmaf(pl_get(g, li), inv_l[g], p);
      const float s_new = (li < n_old ? a.score[row0 + li] : 0.f) + p;
      if (li < n_old || !evict) a.score[row0 + li] = s_new;          // the new token's score is placed with its row
      else s_new_score = s_new;
      const int pz = li < n_old ? a.pos[row0 + li] : t_pos;
      if (evict && pz >= Tn && pz <= t_pos - M) {                      // lowest score, ties -> latest position
        const unsigned long long key = ((unsigned long long)float_ord(s_new) << 32) | (uint32_t)(0x7fffffff - pz);
        if (key < my_min) { my_min = key; my_min_li = li; }
      }
    }
    if (evict) block_arg_extreme<true, CW>(my_min, my_min_li, s_key, s_li, &s_best_key, &s_best_li);
    consumer_sync<CW>();
  }
  // ---- victim (Eq. 7-8); its cosine with every other row (Eq. 9): from the guess, or from a second look at the keys;
  // tau_t (Eq. 10), merged key (Eq. 11-12)
  int vic_li = -1, nn_li = -1;
  bool merge = false, nn_is_new = false;
  float w_e = 0.f, w_c = 1.f, rn_slot = 0.f;
  uint4 kslot = knew;                                                // what goes into the victim's key row
  if (evict) {
    vic_li = s_best_li;
    if (s_best_key == ~0ull) {
      // nothing may be evicted (S_l < T + M): report, drop the new token, keep the cache as it is.  The producer
      // still delivers the value pass; it is drained without being used.
      if (tid == 0) report_error(a.status, D2O_ERR_STATE, 0xDEC00000u | (uint32_t)(sl & 0xfffff));
      for (int s = 0; s < n_st; ++s, ring_next(slot, ph, NS)) {
        stage_wait(&s_full[slot], ph, &s_timeout, a.wait_ns);
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_empty[slot]);
      }
      return;
    }
    if (!D2O_GUARD(vic_li >= 0 && vic_li <= n_old, a.status, 0xC4EC0011u)) vic_li = n_old;
    const float vic_rn = vic_li < n_old ? a.rnorm[row0 + vic_li] : s_new_rn;
    float kvic[EPV];
    Elem<T>::unpack(ld_global_v4((vic_li < n_old ? kpool + (row0 + vic_li) * D : k_new) + lig * EPV), kvic);
    unsigned long long best = 0ull; int best_li = -1;
    int hit = -1;
#pragma unroll
    for (int c = 0; c < NC; ++c) if (cand_li[c] == vic_li) hit = c;
    if (hit >= 0) {
#pragma unroll
      for (int c = 0; c < NC; ++c) if (hit == c) { best = cbest[c]; best_li = cbest_li[c]; }
    } else {
      // The victim was not among the guessed rows (or is the new token itself): the keys once more, straight from
      // global memory.  One row per group of LPR lanes.
      if (tid == 0) atomicAdd(&a.counters[kCntGuessMisses], 1ull);
      for (int li = grp; li < n_old; li += NGRP) {
        float f[EPV];
        Elem<T>::unpack(ld_global_v4(kpool + (row0 + li) * D + lig * EPV), f);
        float x = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) x = fmaf(kvic[e], f[e], x);
        x = group_sum<LPR>(x, gmask);
        if (lig == 0 && li != vic_li) {                              // max similarity, ties -> earliest position
          const unsigned long long key = ((unsigned long long)sim_ord(x * vic_rn * a.rnorm[row0 + li]) << 32) |
                                         (uint32_t)(0x7fffffff - a.pos[row0 + li]);
          if (key > best) { best = key; best_li = li; }
        }
      }
      if (grp == 0 && vic_li != n_old) {                             // the new token as a merge target
        float f[EPV];
        Elem<T>::unpack(knew, f);
        float x = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) x = fmaf(kvic[e], f[e], x);
        x = group_sum<LPR>(x, gmask);
        const unsigned long long key = ((unsigned long long)sim_ord(x * vic_rn * s_new_rn) << 32) | (uint32_t)(0x7fffffff - t_pos);
        if (lig == 0 && key > best) { best = key; best_li = n_old; }
      }
    }
    block_arg_extreme<false, CW>(best, best_li, s_key, s_li, &s_best_key, &s_best_li);
    consumer_sync<CW>();
    nn_li = s_best_li;
    const float mx = ord_float((uint32_t)(s_best_key >> 32));
    const float tau_new = a.beta * mx + (1.0f - a.beta) * tau_old;
    const float thr = isnan(a.tau_override) ? tau_new : a.tau_override;
    merge = mx >= thr && nn_li >= 0;
    if (!D2O_GUARD(nn_li >= 0 && nn_li <= n_old && nn_li != vic_li, a.status, 0xC4EC0012u)) merge = false;
    nn_is_new = (nn_li == n_old);
    const float ew = expf(mx);
    w_e = a.average ? 0.5f : ew / (ew + kEuler);
    w_c = a.average ? 0.5f : kEuler / (ew + kEuler);
    if (tid == 0) {
      a.tau[sidx] = tau_new;
      atomicAdd(&a.counters[kCntDecodeSteps], 1ull);
      atomicAdd(&a.counters[kCntEvictions], 1ull);
      atomicAdd(&a.counters[merge ? kCntMerges : kCntDiscards], 1ull);
    }
    rn_slot = s_new_rn;
    if (warp == 0 && lane < LPR) {
      // keys are not read any more in this launch: merged key row in place, the new token's key into the victim's row
      if (merge) {
        float fk[EPV];
        Elem<T>::unpack(nn_is_new ? knew : ld_global_v4(kpool + (row0 + nn_li) * D + lane * EPV), fk);
#pragma unroll
        for (int e = 0; e < EPV; ++e) fk[e] = w_c * fk[e] + w_e * kvic[e];
        const uint4 kn = Elem<T>::pack(fk);
        Elem<T>::unpack(kn, fk);                                     // norm of what is stored
        float ss = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) ss = fmaf(fk[e], fk[e], ss);
        ss = group_sum<LPR>(ss, gmask);
        const float rnew = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
        if (nn_is_new) { kslot = kn; rn_slot = rnew; }
        else {
          *reinterpret_cast<uint4*>(kpool + (row0 + nn_li) * D + lane * EPV) = kn;
          if (lane == 0) a.rnorm[row0 + nn_li] = rnew;
        }
      }
      if (vic_li != n_old) {
        *reinterpret_cast<uint4*>(kpool + (row0 + vic_li) * D + lane * EPV) = kslot;
        if (lane == 0) {
          a.pos[row0 + vic_li] = t_pos;
          a.score[row0 + vic_li] = s_new_score;
          a.rnorm[row0 + vic_li] = rn_slot;
        }
      }
    }
  }
  // ---- pass V: un-normalised outputs; the value rows of the victim and of the neighbour are picked out of the stream
  if constexpr (kTensor) {
    // out^T (d x heads) = V^T (d x rows) P (rows x heads) on mma.sync.  A stage holds NH = ROWB / 128 column halves
    // of SR rows x 128 bytes, each swizzled (16-byte chunk c of row r sits at chunk c ^ (r & 7)).  Warp w takes the
    // 16 rows rt = w / NH of half hf = w % NH: four 16 x 16 tiles of V^T, read with transposing matrix loads; the
    // weights are split into two 16-bit terms so that the products keep fp32-like accuracy.  The new token is not in
    // the stream: its term is added in the final reduction.
    constexpr int NH = ROWB / 128;
    const int hf = warp % NH, rt = warp / NH;
    float acc[4][4];
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mt][e] = 0.f;
    // per-lane constants: byte offsets of the four transposing loads inside a stage, the weights of head gid
    // (lanes with gid >= G read head 0: their columns of the product are never used)
    const int krow = (lane & 7) + ((lane >> 4) & 1) * 8;             // this lane's row of the 16 x 16 tile for ldmatrix
    const uint32_t tile_off = (uint32_t)(hf * SR * 128 + rt * 16 * 128);
    uint32_t ld_off[4];
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
      ld_off[mt] = tile_off + (uint32_t)(krow * 128 + (((mt * 2 + ((lane >> 3) & 1)) ^ (lane & 7)) << 4));
    const uint32_t ring_u32 = smem_u32(ring);
    const int gw = gid < G ? gid : 0;
    const float* wrow = pl + (size_t)gw * a.row_cap + rt * 16 + 2 * tig;
    const int n_fast = min(n_old, a.row_cap);                       // rows with nothing special about them
    const int vic_row = vic_li < n_old ? vic_li : -64, nn_row = nn_li < n_old ? nn_li : -64;
    int li0 = rt * 16;                                               // first row of this warp's tile
    for (int s = 0; s < n_st; ++s, ring_next(slot, ph, NS), li0 += SR, wrow += SR) {
      stage_wait(&s_full[slot], ph, &s_timeout, a.wait_ns);
      const uint32_t stage_u32 = ring_u32 + (uint32_t)slot * (uint32_t)kStageBytes;
      if (li0 < n_old) {
        uint32_t bh0, bl0, bh1, bl1;
        if (li0 + 16 <= n_fast) {
          const float2 w0 = *reinterpret_cast<const float2*>(wrow), w1 = *reinterpret_cast<const float2*>(wrow + 8);
          split_pair<T>(w0.x, w0.y, bh0, bl0);
          split_pair<T>(w1.x, w1.y, bh1, bl1);
        } else {
          // the last rows of the cache, or rows whose weights are in global memory
          uint4* tile = reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(ring) + (size_t)slot * kStageBytes + tile_off);
          if (li0 + 16 > n_old) {
            // rows past the cache (the slice's padding, the next slice, or nothing at all) count as zero
            for (int i = lane; i < 16 * 8; i += 32)
              if (li0 + (i >> 3) >= n_old) tile[i] = make_uint4(0, 0, 0, 0);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
          }
          const int r0 = li0 + 2 * tig;
          float2 w0, w1;
          w0.x = r0 < n_old ? pl_get(gw, r0) : 0.f;
          w0.y = r0 + 1 < n_old ? pl_get(gw, r0 + 1) : 0.f;
          w1.x = r0 + 8 < n_old ? pl_get(gw, r0 + 8) : 0.f;
          w1.y = r0 + 9 < n_old ? pl_get(gw, r0 + 9) : 0.f;
          split_pair<T>(w0.x, w0.y, bh0, bl0);
          split_pair<T>(w1.x, w1.y, bh1, bl1);
        }
        if ((unsigned)(vic_row - li0) < 16u || (unsigned)(nn_row - li0) < 16u) {
          const uint4* tile = reinterpret_cast<const uint4*>(reinterpret_cast<unsigned char*>(ring) + (size_t)slot * kStageBytes + tile_off);
          if ((unsigned)(vic_row - li0) < 16u && lane < 8) {
            const int r = vic_row - li0;
            stash[hf * 8 + lane] = tile[r * 8 + (lane ^ (r & 7))];
          }
          if ((unsigned)(nn_row - li0) < 16u && lane < 8) {
            const int r = nn_row - li0;
            stash[LPR + hf * 8 + lane] = tile[r * 8 + (lane ^ (r & 7))];
          }
        }
        uint32_t fa[4][4];
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) ldmatrix_x4_trans(stage_u32 + ld_off[mt], fa[mt][0], fa[mt][1], fa[mt][2], fa[mt][3]);
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) mma_16x8x16<T>(acc[mt], fa[mt][0], fa[mt][1], fa[mt][2], fa[mt][3], bh0, bh1);
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) mma_16x8x16<T>(acc[mt], fa[mt][0], fa[mt][1], fa[mt][2], fa[mt][3], bl0, bl1);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_empty[slot]);
    }
    // a victim or neighbour that is the new token itself
    if (grp == 0) {
      if (vic_li == n_old) stash[lig] = vnew;
      if (nn_li == n_old) stash[LPR + lig] = vnew;
    }
    consumer_sync<CW>();                                                 // the ring is drained: reuse it
    // red[rt][g][d]; acc[mt] = (d = hf 64 + mt 16 + gid, + 8) x (heads 2 tig, 2 tig + 1)
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int g = 2 * tig + (e & 1), dd = hf * 64 + mt * 16 + gid + (e >> 1) * 8;
        if (g < G) red[((size_t)rt * G + g) * D + dd] = acc[mt][e];
      }
    consumer_sync<CW>();
    for (int i = tid; i < G * D; i += kConsThreads) {
      float t = pl_get(i / D, n_old) * Elem<T>::to_float(v_new[i % D]);
#pragma unroll
      for (int w = 0; w < kConsWarps / NH; ++w) t += red[(size_t)w * G * D + i];
      out[(size_t)sl * G * D + i] = Elem<T>::from_float(t * inv_l[i / D]);
    }
  } else {
    float acc[G][EPV];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
      for (int e = 0; e < EPV; ++e) acc[g][e] = 0.f;
    for (int s = 0; s < n_st; ++s, ring_next(slot, ph, NS)) {
      stage_wait(&s_full[slot], ph, &s_timeout, a.wait_ns);
      const uint4* st = ring + (size_t)slot * SR * LPR + (size_t)grp * LPR + lig;
      const int lbase = s * SR + grp;                                // this thread's rows: lbase + u * NGRP
      // a plain stage: all rows are cache rows with their weights in shared memory, neither victim nor neighbour
      const bool plain = (s + 1) * SR <= n_plain_fma && (unsigned)(vic_li - s * SR) >= (unsigned)SR &&
                         (unsigned)(nn_li - s * SR) >= (unsigned)SR;
      if (plain) {
        uint4 raw[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) raw[u] = st[(size_t)u * NGRP * LPR];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          float f[EPV];
          Elem<T>::unpack(raw[u], f);
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const float p = pl[(size_t)g * a.row_cap + lbase + u * NGRP];
#pragma unroll
            for (int e = 0; e < EPV; e += 2) {
              const float2 r = ffma2(make_float2(p, p), make_float2(f[e], f[e + 1]), make_float2(acc[g][e], acc[g][e + 1]));
              acc[g][e] = r.x; acc[g][e + 1] = r.y;
            }
          }
        }
      } else {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int li = lbase + u * NGRP;
          if (li < n) {
            const uint4 raw = st[(size_t)u * NGRP * LPR];
            if (li == vic_li) stash[lig] = raw;
            if (li == nn_li) stash[LPR + lig] = raw;
            float f[EPV];
            Elem<T>::unpack(raw, f);
#pragma unroll
            for (int g = 0; g < G; ++g) {
              const float p = pl_get(g, li);
#pragma unroll
              for (int e = 0; e < EPV; e += 2) {
                const float2 r = ffma2(make_float2(p, p), make_float2(f[e], f[e + 1]), make_float2(acc[g][e], acc[g][e + 1]));
                acc[g][e] = r.x; acc[g][e + 1] = r.y;
              }
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_empty[slot]);
    }
    // combine the row groups of a warp, then the warps
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
      for (int g = 0; g < G; ++g)
#pragma unroll
        for (int e = 0; e < EPV; ++e) acc[g][e] += __shfl_xor_sync(0xffffffffu, acc[g][e], o);
    }
    consumer_sync<CW>();                                                 // the ring is drained: reuse it
    if (lane < LPR) {
#pragma unroll
      for (int g = 0; g < G; ++g)
#pragma unroll
        for (int e = 0; e < EPV; ++e) red[((size_t)warp * G + g) * D + lane * EPV + e] = acc[g][e];
    }
    consumer_sync<CW>();
    for (int i = tid; i < G * D; i += kConsThreads) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < kConsWarps; ++w) t += red[(size_t)w * G * D + i];
      out[(size_t)sl * G * D + i] = Elem<T>::from_float(t * inv_l[i / D]);
    }
  }
  if (tid == 0 && s_timeout == 2) report_error(a.status, D2O_ERR_TIMEOUT, 0xDEC10000u | (uint32_t)(sl & 0xffff));
  // This warp's part of the slice's state is complete.  When a chained step follows, the producer warp waits for
  // every consumer warp's arrival and publishes the slice's step counter.  The next step's CTA reads the rows,
  // positions and norms that warp 0 writes last with bulk copies, hence the proxy fence in that warp.
  auto consumer_done = [&]() {
    if (a.publish) {
      if (warp == 0) asm volatile("fence.proxy.async.global;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_done);
    }
  };
  if (!evict) {
    // the cache is not full yet: append the new token's row
    if (grp == 0) {
      *reinterpret_cast<uint4*>(kpool + (row0 + n_old) * D + lig * EPV) = knew;
      *reinterpret_cast<uint4*>(vpool + (row0 + n_old) * D + lig * EPV) = vnew;
      if (lig == 0) { a.pos[row0 + n_old] = t_pos; a.rnorm[row0 + n_old] = s_new_rn; }
    }
    if (tid == 0) {
      a.len[sidx] = n;
      atomicAdd(&a.counters[kCntDecodeSteps], 1ull);
    }
    consumer_done();
    return;
  }
  // ---- merged value row (Eq. 11); the new token's value takes the victim's row
  if (warp == 0 && lane < LPR) {
    uint4 vslot = vnew;
    if (merge) {
      float fv[EPV], vv[EPV];
      Elem<T>::unpack(stash[LPR + lane], fv);                        // the neighbour's value row (the new token's if it is the neighbour)
      Elem<T>::unpack(stash[lane], vv);                              // the victim's value row
#pragma unroll
      for (int e = 0; e < EPV; ++e) fv[e] = w_c * fv[e] + w_e * vv[e];
      const uint4 vn = Elem<T>::pack(fv);
      if (nn_is_new) vslot = vn;
      else *reinterpret_cast<uint4*>(vpool + (row0 + nn_li) * D + lane * EPV) = vn;
    }
    if (vic_li != n_old) *reinterpret_cast<uint4*>(vpool + (row0 + vic_li) * D + lane * EPV) = vslot;
  }
  consumer_done();
}

// ------------------------------------------------------------------------------------ launch
// ring stages (each with the 1/|k| and position slots of its rows), probabilities, stash
static size_t stage_bytes(int cw, int row_bytes) { return (size_t)stage_bytes_of(cw) + 2 * (size_t)(stage_bytes_of(cw) / row_bytes) * 4; }
// ring stages (each with the 1/|k| and position slots of its rows), probabilities, stash
static size_t smem_bytes(int cw, int row_cap, int stages, int G, int row_bytes) {
  return (size_t)stages * stage_bytes(cw, row_bytes) + (size_t)G * row_cap * 4 + 2 * (size_t)row_bytes;
}

template <typename T, int D, int G, int CW, int OCC = 0>
static cudaError_t launch_one(const DecodeArgs& a, const CUtensorMap& map_k, const CUtensorMap& map_v, int n_slices,
                              const void* q, const void* k, const void* v, void* out, void* kpool, void* vpool,
                              cudaStream_t st, bool overlap_previous) {
  const size_t smem = smem_bytes(CW, a.row_cap, a.stages, G, D * (int)sizeof(T));
  auto kern = decode_kernel<T, D, G, CW, OCC>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)n_slices); cfg.blockDim = dim3((CW + 1) * 32); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = overlap_previous ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, a, map_k, map_v, (const T*)q, (const T*)k, (const T*)v, (T*)out, (T*)kpool, (T*)vpool);
}

// G = 1, 2: 4, 8 or 16 consumer warps; G = 4, 8: the same
#define D2O_LAUNCH(GG, CC) launch_one<T, D, GG, CC>(a, map_k, map_v, n_slices, q, k, v, out, kpool, vpool, st, overlap)
template <typename T, int D>
static cudaError_t launch_g(int G, int cw, const DecodeArgs& a, const CUtensorMap& map_k, const CUtensorMap& map_v, int n_slices,
                            const void* q, const void* k, const void* v, void* out, void* kpool, void* vpool,
                            cudaStream_t st, bool overlap, bool three_per_sm) {
  // grouped queries on the tensor path with eight warps: a second build capped at 72 registers for three CTAs per SM
  if constexpr (sizeof(T) == 2) {
    if (three_per_sm && cw == 8 && G == 4)
      return launch_one<T, D, 4, 8, 3>(a, map_k, map_v, n_slices, q, k, v, out, kpool, vpool, st, overlap);
    if (three_per_sm && cw == 8 && G == 8)
      return launch_one<T, D, 8, 8, 3>(a, map_k, map_v, n_slices, q, k, v, out, kpool, vpool, st, overlap);
  }
  switch (G) {
    case 1: return cw == 16 ? D2O_LAUNCH(1, 16) : cw == 4 ? D2O_LAUNCH(1, 4) : D2O_LAUNCH(1, 8);
    case 2: return cw == 16 ? D2O_LAUNCH(2, 16) : cw == 4 ? D2O_LAUNCH(2, 4) : D2O_LAUNCH(2, 8);
    case 4: return cw == 16 ? D2O_LAUNCH(4, 16) : cw == 4 ? D2O_LAUNCH(4, 4) : D2O_LAUNCH(4, 8);
    default: return cw == 16 ? D2O_LAUNCH(8, 16) : cw == 4 ? D2O_LAUNCH(8, 4) : D2O_LAUNCH(8, 8);
  }
}
#undef D2O_LAUNCH

// CTAs per SM the registers allow (mirrors the kernel's __launch_bounds__)
static int max_per_sm(int cw, int G, int elem_size) { return ctas_per_sm(cw, G, elem_size); }

// Ring depth for `max_rows` rows per slice when `per_sm` CTAs are to share an SM.  false if the per-row arrays leave
// no room for a ring.  Occupancy matters more than depth: measured on the 7B-shaped stack with caches of 700 to
// 1900 rows, three CTAs with two stages each beat two CTAs with three or four stages (108 us vs 113 us per step).
static bool plan_tier(int cw, int smem_rows, int row_bytes, int G, int D, int per_sm, int* row_cap, int* stages_out) {
  const long sm_total = 227 * 1024;
  const int cap = (smem_rows + 7) & ~7;
  const int min_stages = max(2, (cw * G * D * 4 + stage_bytes_of(cw) - 1) / stage_bytes_of(cw));   // the ring doubles as `red`
  const long fixed = (long)G * cap * 4 + 2L * row_bytes + 2048;                               // + static shared memory
  const long room = sm_total / per_sm - 1024 - fixed;
  const int fit = room > 0 ? (int)(room / (long)stage_bytes(cw, row_bytes)) : 0;
  if (fit < min_stages) return false;
  *row_cap = cap;
  *stages_out = max(min_stages, min(fit, per_sm == 1 ? 6 : (per_sm == 2 ? 4 : (per_sm == 3 ? 3 : 2))));
  return true;
}

// Best occupancy tier that fits `max_rows`; 0 = none.
static int best_tier(int cw, int smem_rows, int row_bytes, int G, int D, int occ, int* row_cap, int* stages) {
  for (int per_sm = occ > 0 ? occ : max_per_sm(cw, G, row_bytes / D); per_sm >= 1; --per_sm)
    if (plan_tier(cw, smem_rows, row_bytes, G, D, per_sm, row_cap, stages)) return per_sm;
  return 0;
}

static bool plan(int cw, int smem_rows, int row_bytes, int G, int D, int want_stages, int occ, int* row_cap, int* stages_out) {
  if (want_stages <= 0) return best_tier(cw, smem_rows, row_bytes, G, D, occ, row_cap, stages_out) != 0;
  const long sm_total = 227 * 1024;
  const int cap = (smem_rows + 7) & ~7;
  const int min_stages = max(2, (cw * G * D * 4 + stage_bytes_of(cw) - 1) / stage_bytes_of(cw));
  const long fixed = (long)G * cap * 4 + 2L * row_bytes + 2048;
  if (want_stages < min_stages || want_stages > kMaxStages) return false;
  if (fixed + (long)want_stages * (long)stage_bytes(cw, row_bytes) > sm_total - 1024) return false;
  *row_cap = cap; *stages_out = want_stages;
  return true;
}

// Rows of a slice whose logits stay in shared memory: all of them while that takes 16 KB or less; else enough for
// slices twice as long as the mean (the budgets of Eq. 5 give a few layers several times the mean, and sizing
// the array for those would cost every CTA its ring depth or the SM a resident CTA).
static int smem_rows_for(int max_rows, double mean_rows, int G) {
  const int free_rows = 16 * 1024 / (4 * G);
  if (max_rows <= free_rows) return max_rows;
  return min(max_rows, max(free_rows, (int)(2.0 * mean_rows)));
}

// `chained`: this step follows another decode step of the same layers on the same stream, and its inputs were
// complete before that one was launched.  Its grids are then launched with programmatic stream serialisation and
// may start while the previous step's last CTAs are still running; every CTA waits for its own slice's step counter
// instead of the whole previous grid.  `publish`: a chained step follows this one, so every CTA writes its slice's
// step counter when the slice's state is complete.
cudaError_t launch_decode(const d2o_ctx* c, int l0, int l1, const void* q, const void* k, const void* v, void* out,
                          cudaStream_t st, d2o_status* why, bool chained, bool publish) {
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
  a.step = c->layer_steps[l0];
  a.plen = (const int32_t*)(S + c->lay.plen);
  a.beta = g.beta; a.tau_override = g.tau_override; a.average = g.merge_policy;
  a.wait_ns = c->wait_limit_us > 0 ? (unsigned long long)c->wait_limit_us * 1000ull : kWaitNs;
  a.stop_stage = c->producer_stop_stage;
  a.pool_rows = c->pool_rows;
  a.steps_done = (int32_t*)(S + c->lay.steps_done);
  a.chained = chained ? 1 : 0;
  a.publish = publish ? 1 : 0;
  a.l2_hints = c->decode_l2_hints;
  const int G = c->group, Hkv = g.n_kv_heads;
  const int row_bytes = g.d_head * c->elem_size;
  void* kpool = S + c->lay.kpool; void* vpool = S + c->lay.vpool;
  // rows of the longest slice of a pair, and the mean over all slices (a cache cannot hold more than was generated)
  const int t_now = g.prompt_len + c->layer_steps[l0];
  int max_rows = 0;
  double sum_rows = 0.0;
  for (int l = l0; l < l1; ++l)
    for (int b = 0; b < B; ++b) {
      max_rows = max(max_rows, min(c->h_pair_max[b * L + l], t_now) + 1);
      sum_rows += (double)min((long long)c->h_pair_sum[b * L + l], (long long)t_now * g.n_kv_heads) / g.n_kv_heads + 1.0;
    }
  // all layers in one call: CTAs take the slices largest cache first, so the long ones do not end up in the tail
  const bool ordered = (l0 == 0 && l1 == L);
  a.order = ordered ? (const int32_t*)(S + c->lay.order) : nullptr;
  a.spill = (float*)(c->scratch + c->slay.pl_spill);
  const int n_pairs = (l1 - l0) * B;
  const double mean_rows = sum_rows / n_pairs;
  auto rows_of_pair = [&](int i) {                                    // i-th pair in launch order: its longest slice
    const int pr = ordered ? c->h_order[i] : (l0 * B + i);
    return min(c->h_pair_max[(pr % B) * L + pr / B], t_now) + 1;
  };

  // A step takes at least as long as its longest slice takes in one CTA, and in a chain of steps a slice's CTAs
  // follow one another.  On the tensor path, where a few layers hold several times the mean budget and an
  // eight-warp CTA streams about 15 GB/s, the longest slices go into a launch of their own with sixteen consumer
  // warps per CTA, and the rest follows in a second launch that is allowed to start while the first is still running
  // (the two share no slice).  Estimate with rough per-row costs of an eight-warp CTA; exactness does not matter,
  // the split only has to catch the outliers.  On the FMA path an eight-warp CTA streams a 2048-row slice in well
  // under a step and the split only costs (measured with and without on the 7B-shaped configs, single and chained
  // steps): one launch.
  int n_long = 0;
  if (ordered && c->decode_warps == 0 && c->decode_long_pairs == 0 && n_pairs > 1 && tensor_path(c->elem_size, G)) {
    const double fixed_us = 8.0, row_us = 0.025;
    const double slots = (double)c->n_sms * ctas_per_sm(8, G, c->elem_size);
    double work = 0.0;
    for (int i = 0; i < n_pairs; ++i) work += Hkv * (fixed_us + row_us * rows_of_pair(i));
    // measured optimum on the long-context config: twelve pairs
    const double limit = 0.55 * work / slots;
    while (n_long < n_pairs && (n_long + 1) * Hkv <= 2 * c->n_sms && fixed_us + row_us * rows_of_pair(n_long) > limit) ++n_long;
    if (n_long == n_pairs) n_long = 0;
  } else if (ordered && c->decode_long_pairs > 0) {
    n_long = min(c->decode_long_pairs, n_pairs - 1);
  }

  // one launch over the pairs [p0, p1) of the order
  auto launch_class = [&](int p0, int p1, int cw, bool overlap) -> cudaError_t {
    int cls_max = 0;
    long long cls_sum = 0;
    for (int i = p0; i < p1; ++i) { const int r = rows_of_pair(i); cls_max = max(cls_max, r); cls_sum += r; }
    const int n_slices = (p1 - p0) * Hkv;
    int row_cap, stages;
    int smem_rows = smem_rows_for(cls_max, (double)cls_sum / (p1 - p0), G);
    if (c->decode_smem_rows > 0) smem_rows = min(cls_max, c->decode_smem_rows);
    // Tensor path, eight warps, G >= 4: three CTAs per SM (a build capped at 72 registers) when three ring stages
    // and the logits of rows up to 1.5 x the mean still fit a third of the shared memory; measured on the
    // 8B-shaped config 382 vs 396 us per step, while with longer slices (two CTAs anyway) that build only spills.
    bool three = false;
    if (tensor_path(c->elem_size, G) && cw == 8 && G >= 4 && c->decode_stages == 0) {
      const long third = 227 * 1024 / 3 - 1024 - 2L * row_bytes - 2048 - 3L * (long)stage_bytes(8, row_bytes);
      const int rows3 = (int)(third / (4 * G)) & ~7;
      if (rows3 >= 1.5 * (double)cls_sum / (p1 - p0) || rows3 >= cls_max) {
        three = true;
        if (c->decode_smem_rows == 0) smem_rows = min(smem_rows, rows3);
      }
    }
    if (!plan(cw, smem_rows, row_bytes, G, g.d_head, c->decode_stages, three ? 3 : 0, &row_cap, &stages)) {
      *why = D2O_ERR_UNSUPPORTED;
      return cudaSuccess;
    }
    c->decode_launches += 1;
    DecodeArgs ac = a;
    ac.row_cap = row_cap; ac.stages = stages; ac.pair_base = p0;
    // 16-bit caches with grouped queries read their rows through tensor maps (swizzled stages)
    CUtensorMap map_k, map_v;
    memset(&map_k, 0, sizeof(map_k));
    memset(&map_v, 0, sizeof(map_v));
    if (tensor_path(c->elem_size, G)) {
      const int box_rows = stage_bytes_of(cw) / row_bytes;
      if (c->pool_rows >= (1ll << 31) || !encode_rows_2d(&map_k, g.dtype, kpool, (uint64_t)c->pool_rows, g.d_head, box_rows) ||
          !encode_rows_2d(&map_v, g.dtype, vpool, (uint64_t)c->pool_rows, g.d_head, box_rows)) {
        *why = D2O_ERR_UNSUPPORTED;
        return cudaSuccess;
      }
    }
    // inputs and outputs of the step are indexed by the slice's place in the call, which the kernel derives itself
    if (g.dtype == D2O_F32)
      return g.d_head == 64 ? launch_g<float, 64>(G, cw, ac, map_k, map_v, n_slices, q, k, v, out, kpool, vpool, st, overlap, three)
                            : launch_g<float, 128>(G, cw, ac, map_k, map_v, n_slices, q, k, v, out, kpool, vpool, st, overlap, three);
    if (g.dtype == D2O_F16)
      return g.d_head == 64 ? launch_g<__half, 64>(G, cw, ac, map_k, map_v, n_slices, q, k, v, out, kpool, vpool, st, overlap, three)
                            : launch_g<__half, 128>(G, cw, ac, map_k, map_v, n_slices, q, k, v, out, kpool, vpool, st, overlap, three);
    return g.d_head == 64 ? launch_g<__nv_bfloat16, 64>(G, cw, ac, map_k, map_v, n_slices, q, k, v, out, kpool, vpool, st, overlap, three)
                          : launch_g<__nv_bfloat16, 128>(G, cw, ac, map_k, map_v, n_slices, q, k, v, out, kpool, vpool, st, overlap, three);
  };

  if (n_long > 0) {
    cudaError_t e = launch_class(0, n_long, 16, chained);
    if (e != cudaSuccess || *why != D2O_OK) return e;
    const int rest = (n_pairs - n_long) * Hkv;
    int rest_max = rows_of_pair(n_long);
    const int cw = (c->decode_warps == 4 || c->decode_warps == 8) ? c->decode_warps
                   : ((G <= 2 && rest >= 8 * c->n_sms * 4 && rest_max <= 2304) ? 4 : 8);
    return launch_class(n_long, n_pairs, cw, true);
  }
  // Consumer warps per CTA.  One head per KV head and enough small slices for seven and more CTAs on every SM:
  // four warps (measured on the serving-shaped config, 8192 slices of ~410 rows: 350 vs 370 us per step; with the
  // upper clamp of the budgets removed, slices up to 2048 rows: 306 vs 348 us chained, 354 vs 350 in single calls,
  // and at 32 sequences 1299 vs 1453 us).
  // Grouped queries with slices several times the mean and few of them: sixteen warps, one CTA per SM, so that the
  // longest slice streams twice as fast.  Otherwise eight.
  const int n_slices = n_pairs * Hkv;
  int cw = c->decode_warps;
  if (cw == 0) {
    cw = 8;
    if (G <= 2 && n_slices >= 8 * c->n_sms * 4 && max_rows <= 2304) cw = 4;
    if (G >= 4 && n_slices <= c->n_sms * 8 && max_rows > 2.0 * mean_rows) cw = 16;
  }
  return launch_class(0, n_pairs, cw, chained);
}

}  // namespace d2o
