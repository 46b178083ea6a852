// Device code of the WeightedKV decode step for sm_100a.
//
// One launch runs one iteration of the paper's Algorithm 1 for every lane (sequence, kv-head) of a layer.
// A lane's slots are cut into n_splits contiguous chunks ("units").  Whoever processes a unit streams its K and V
// rows through a shared-memory ring filled by bulk asynchronous copies (one producer thread, mbarrier completion),
// computes the logits, and keeps an online-softmax partial of the attention output.  When all units of a lane are
// done, the partials become o_t, the logits become the probabilities A_t (reproducible binary32 arithmetic below),
// A_t is folded into the accumulated scores, the eviction victim is picked, its value is merged into the right
// neighbour and the slot bookkeeping is relinked.  Two schedules share that code:
//
//   scan_kernel + lane_epilogue_kernel   any split count, two launches.  One short-lived CTA per unit parks logits
//                               and its partial in global scratch; a second kernel with one CTA per lane finishes
//                               the lanes.  Keeps HBM busiest when there are many lanes.
//   decode_step_cluster_kernel           one launch: the n_splits CTAs of a lane form one thread-block cluster (n_splits in {1,2,4,8,16}).
//                               Logits stay in shared memory, partials are read through distributed shared memory
//                               and every CTA folds its own slots.  Best when there are few lanes (latency-bound).
//
// Slots are not kept in position order.  A lane owns budget+1 slots; each holds one cache entry
// (K row, V row, accumulated score a, original position pos) and is chained to its position neighbours
// through next/prev, so "the right adjacent entry" of Algorithm 1 is next[j] and freeing an entry never
// moves cache rows.  n of Algorithm 1 is not stored: n_i = t - pos_i + 1.
//
// Reproducible binary32 score path (decides the eviction index, therefore specified operation by operation;
// all operations IEEE round-to-nearest-even, explicit intrinsics so the compiler neither contracts nor
// reassociates):
//   dot   : 16 partial sums over contiguous channel blocks of head_dim/16; inside a block the even channels and the
//           odd channels each form an fma chain from +0 (one packed fp32x2 fma per channel pair) and the two chains
//           are added; then a butterfly p_r + p_{r^off}, off = 8,4,2,1; logit = scale * p.
//   exp   : 0 below -87; n = rint(x*LOG2E); Cody-Waite reduction with LN2_HI/LN2_LO; degree-7 Taylor
//           polynomial in Horner form with fma; exact scaling by 2^n.
//   sum   : Z = float(sum_i trunc(e_i * 2^40)) * 2^-40 -- an integer sum, hence order-free.
//   prob  : e_i / Z; group mean (((p0+p1)+p2)+...)*(1/G); a += pbar; abar = a / float(n).
//   pick  : minimum of (abar, pos) lexicographically == minimum of (bits(abar) << 32 | pos).
//   merge : D = abar_j + abar_r; w_j = abar_j/D; w_r = abar_r/D; v = fma(w_j, v_j, w_r*v_r), rounded to T.
// The attention output o_t is not part of that chain and uses fast exp2 with an online softmax.
#pragma once
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace wkv {

#ifndef WKV_RING_BYTES
#define WKV_RING_BYTES 32768          // shared-memory ring per CTA (K and V tiles, all stages)
#endif
constexpr int kTileSlots = 32;        // cache entries per pipeline stage
constexpr int kConsumerWarps = 4;     // each owns 8 rows of a tile
constexpr int kThreads = (kConsumerWarps + 1) * 32;   // + one producer warp
constexpr int kMaxSplits = 64;
constexpr uint32_t kSpinLimit = 1u << 22;             // polls of a bounded wait (mbarrier, or a lane's arrival counter; each poll sleeps briefly)

enum StatusBits : uint32_t { kStatusWaitTimeout = 1u, kStatusBadLink = 2u };

// lane_state[lane][8]
enum { LS_LEN = 0, LS_T = 1, LS_HEAD = 2, LS_TAIL = 3, LS_FREE = 4, LS_STRIDE = 8 };

struct StepParams {
  void* Kc;              // [lanes_total][cap][D] storage type
  void* Vc;
  float* a;              // [lanes_total][cap]
  int32_t* pos;          // [lanes_total][cap]
  int32_t* next;         // [lanes_total][cap]
  int32_t* prev;         // [lanes_total][cap]
  int32_t* lane_state;   // [lanes_total][LS_STRIDE]
  float* logits;         // scratch [lanes_per_layer*G][cap]
  float* part;           // scratch [lanes_per_layer][n_splits][G][D+2] : m, l, o[D] per unit / piece of a lane
  uint32_t* ticket;      // scratch [lanes_per_layer] or nullptr: units of the lane whose scan is finished (zero between calls)
  uint32_t* status;      // device status word
  const void* q;         // [B][..][Hq][D]   batch stride q_bs elements
  const void* k;         // [B][..][Hkv][D]  batch stride kv_bs elements
  const void* v;
  void* out;             // batch stride out_bs elements
  int32_t* evicted;      // or nullptr; batch stride ev_bs
  float* probs;          // or nullptr; [B][Hq][budget+1]
  const int32_t* seq_lens;   // or nullptr
  long long q_bs, kv_bs, out_bs, ev_bs;
  int tok_idx;           // index of this token inside the prefill call (activity test against seq_lens)
  int lane0;             // first global lane of this layer
  int n_kv_heads;
  int cap;               // slots per lane (>= budget+1, multiple of 4)
  int budget, window, sink;
  int n_splits;          // units per lane (even deal); with the flat deal: the most pieces a lane can have
  int flat_chunk;        // 0: even deal, CTA = (lane, unit).  c > 0: flat deal, CTA i takes tiles [i*c, (i+1)*c) of all lanes' tiles
  int tiles_cap;         // flat deal: tiles per lane in that sequence = ceil((budget + 1) / 32)
  int n_lanes;           // lanes of this launch
  int chunk_cap;         // cluster kernel: logits one CTA can hold per query head (its tiles * 32)
  int merge;
  int wait_at_start;     // scan kernel: how it orders itself against the preceding kernel, 0 / 1 / 2 (see scan_kernel)
  int ep_stage_slots;    // lane epilogue kernel: entries of a and pos its dynamic shared memory can stage (0: none)
  // Where the lane epilogue finds its logits and puts the optional probabilities: logits of query head g of lane x at
  // logits[(x * logit_rows + logit_row0 + g) * cap + slot], probabilities at probs[(x * probs_rows + probs_row0 + g) *
  // probs_stride + slot].  A decode step has logit_rows = probs_rows = G, row0 = 0, probs_stride = budget + 1.
  int logit_rows, logit_row0, probs_rows, probs_row0, probs_stride;
  // Blocked prompt tail (wkv_block.cuh): this launch finishes token number block_step of a block of block_tokens tokens
  // (0: not a blocked tail) whose logits against the cache as it was before the block were parked by one sweep.
  int block_tokens, block_step;
  int block_n;           // lane_epilogue_block_kernel: tokens of the block that this one launch finishes, one after the other
  long long kv_ts;       // ... elements between consecutive tokens' k (and v) rows of one sequence
  long long ev_ts;       // ... int32 entries between consecutive tokens' removed positions (0: one shared entry)
  const float* lgx;      // [lanes][logit_rows][block_tokens]: logits against the block's own keys (entries that joined inside the block)
  float* rec_rows;       // [lanes][2 * block_tokens][D] fp32: value rows as they were before a step of the block changed them
  int32_t* rec_slot;     // [lanes][2 * block_tokens]: their slots (entry 2*step: the removed entry, 2*step + 1: its right neighbour), -1 = none
  float scale;
  // Tensor map over the value cache as a [lanes_total * cap][D] matrix: boxes of 64 elements x 32 rows, 128-byte
  // swizzle.  Encoded by the host for configurations whose scan takes its V tiles that way (Cfg::kMmaPV), else unused.
  alignas(64) unsigned char vmap[128];
};

// ------------------------------------------------------------------------------------------------
// small PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `limit` polls, records it in the status word and returns false.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t* status, uint32_t limit = kSpinLimit) {
  for (uint32_t it = 0; it < limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 64) __nanosleep(64);
  }
  atomicOr(status, kStatusWaitTimeout);
  return false;
}
// A consumer warp hands a ring stage back to the producer.  The fence puts every lane's reads of the stage ahead of
// lane 0's arrival whatever instruction did the reading: with fragment loads (ldmatrix) in place of plain loads, the
// reads of a tile's last channels were observed behind the arrival, picking up the tile that the producer put there next.
__device__ __forceinline__ void release_stage(uint64_t* empty_bar) {
  __threadfence_block();
  __syncwarp();
  if ((threadIdx.x & 31) == 0) mbar_arrive(empty_bar);
}
// Bulk asynchronous copy global -> this CTA's shared memory, completion counted in bytes on an mbarrier.
// dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void bulk_g2s_hint(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
               : "memory");
}
// Tiled tensor-map copy global -> this CTA's shared memory: the box of `tmap` whose first element is (x, y) = (element
// in the row, row).  x * element size must be a multiple of 16 bytes; dst 128-byte aligned (1024 for swizzled boxes).
__device__ __forceinline__ void tensor_g2s_2d(void* dst, const void* tmap, int x, int y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
                   smem_u32(dst)),
               "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar))
               : "memory");
}
// The same copy with an L2 eviction-priority policy (from l2_policy_evict_first) for data that is streamed.
__device__ __forceinline__ void tensor_g2s_2d_hint(void* dst, const void* tmap, int x, int y, uint64_t* bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(
          smem_u32(dst)),
      "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
// Hint: bring [src, src + bytes) into L2.  src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void l2_prefetch(const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
// Programmatic dependent launch.  griddep_wait: block until the kernel this one was launched behind has completed and
// its writes are visible (returns at once when the launch carried no such dependency).  griddep_launch: allow the
// next kernel in the stream to begin once every CTA of this grid has called it or exited.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Barrier among the first NT threads of the CTA (NT = kThreads: the whole CTA).
template <int NT>
__device__ __forceinline__ void group_sync() {
  if constexpr (NT == kThreads) __syncthreads();
  else asm volatile("bar.sync 1, %0;" ::"n"(NT) : "memory");
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ------------------------------------------------------------------------------------------------
// storage-type helpers: a lane's EPL = D/16 contiguous channels of a row, widened to fp32
// ------------------------------------------------------------------------------------------------
template <int EPL>
__device__ __forceinline__ void load_chunk(const float* p, float (&x)[EPL]) {
#pragma unroll
  for (int i = 0; i < EPL; i += 4) {
    float4 t = *reinterpret_cast<const float4*>(p + i);
    x[i] = t.x; x[i + 1] = t.y; x[i + 2] = t.z; x[i + 3] = t.w;
  }
}
template <int EPL>
__device__ __forceinline__ void load_chunk(const __nv_bfloat16* p, float (&x)[EPL]) {
  if constexpr (EPL == 4) {
    uint2 t = *reinterpret_cast<const uint2*>(p);
    x[0] = __uint_as_float(t.x << 16); x[1] = __uint_as_float(t.x & 0xffff0000u);
    x[2] = __uint_as_float(t.y << 16); x[3] = __uint_as_float(t.y & 0xffff0000u);
  } else {
#pragma unroll
    for (int i = 0; i < EPL; i += 8) {
      uint4 t = *reinterpret_cast<const uint4*>(p + i);
      x[i + 0] = __uint_as_float(t.x << 16); x[i + 1] = __uint_as_float(t.x & 0xffff0000u);
      x[i + 2] = __uint_as_float(t.y << 16); x[i + 3] = __uint_as_float(t.y & 0xffff0000u);
      x[i + 4] = __uint_as_float(t.z << 16); x[i + 5] = __uint_as_float(t.z & 0xffff0000u);
      x[i + 6] = __uint_as_float(t.w << 16); x[i + 7] = __uint_as_float(t.w & 0xffff0000u);
    }
  }
}
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Packed pairs of binary32 values in one 64-bit register.  fma2 / mul2 are two independent IEEE round-to-nearest
// operations per instruction (no flush-to-zero), so each half is bit-identical to the scalar fma / multiply.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ float lo_of(f32x2 v) { return __uint_as_float((uint32_t)v); }
__device__ __forceinline__ float hi_of(f32x2 v) { return __uint_as_float((uint32_t)(v >> 32)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// NPAIR (even, odd) channel pairs of a row chunk, widened to fp32.  16-byte aligned except the 8-byte bf16 x 4 case.
template <int NPAIR>
__device__ __forceinline__ void load_pairs(const float* p, f32x2 (&x)[NPAIR]) {
#pragma unroll
  for (int i = 0; i < NPAIR; i += 2) {
    const float4 t = *reinterpret_cast<const float4*>(p + 2 * i);
    x[i] = pack2(t.x, t.y);
    x[i + 1] = pack2(t.z, t.w);
  }
}
template <int NPAIR>
__device__ __forceinline__ void load_pairs(const __nv_bfloat16* p, f32x2 (&x)[NPAIR]) {
  if constexpr (NPAIR == 2) {
    const uint2 t = *reinterpret_cast<const uint2*>(p);
    x[0] = pack2(__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xffff0000u));
    x[1] = pack2(__uint_as_float(t.y << 16), __uint_as_float(t.y & 0xffff0000u));
  } else {
#pragma unroll
    for (int i = 0; i < NPAIR; i += 4) {
      const uint4 t = *reinterpret_cast<const uint4*>(p + 2 * i);
      x[i + 0] = pack2(__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xffff0000u));
      x[i + 1] = pack2(__uint_as_float(t.y << 16), __uint_as_float(t.y & 0xffff0000u));
      x[i + 2] = pack2(__uint_as_float(t.z << 16), __uint_as_float(t.z & 0xffff0000u));
      x[i + 3] = pack2(__uint_as_float(t.w << 16), __uint_as_float(t.w & 0xffff0000u));
    }
  }
}

// Tensor-core pieces of the P.V half for four query heads (bf16 rows).  D[16x8] += A[16x8] * B[8x8], fp32 accumulate.
__device__ __forceinline__ void mma_m16n8k8_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5}, {%6}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(b0));
}
// Four transposed 8x8 bf16 matrices; lanes 8i..8i+7 give the row addresses of matrix i (16 bytes each, shared memory).
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* row_addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_u32(row_addr))
               : "memory");
}
__device__ __forceinline__ uint32_t bf16_bits(__nv_bfloat16 x) { return (uint32_t)__bfloat16_as_ushort(x); }

// ------------------------------------------------------------------------------------------------
// reproducible exp (see the header comment)
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float repro_exp(float x) {
  if (x < -87.0f) return 0.0f;
  const float LOG2E = __uint_as_float(0x3fb8aa3bu);
  const float NLN2_HI = -__uint_as_float(0x3f317000u);
  const float NLN2_LO = -__uint_as_float(0x3805fdf4u);
  const float n = rintf(__fmul_rn(x, LOG2E));
  float f = __fmaf_rn(n, NLN2_HI, x);
  f = __fmaf_rn(n, NLN2_LO, f);
  float r = __uint_as_float(0x39500d01u);                  // 1/5040
  r = __fmaf_rn(r, f, __uint_as_float(0x3ab60b61u));       // 1/720
  r = __fmaf_rn(r, f, __uint_as_float(0x3c088889u));       // 1/120
  r = __fmaf_rn(r, f, __uint_as_float(0x3d2aaaabu));       // 1/24
  r = __fmaf_rn(r, f, __uint_as_float(0x3e2aaaabu));       // 1/6
  r = __fmaf_rn(r, f, 0.5f);
  r = __fmaf_rn(r, f, 1.0f);
  r = __fmaf_rn(r, f, 1.0f);
  return __fmul_rn(r, __int_as_float(((int)n + 127) << 23));
}

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long x) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
  return x;
}
__device__ __forceinline__ unsigned long long warp_min_u64(unsigned long long x) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    unsigned long long y = __shfl_xor_sync(0xffffffffu, x, off);
    x = y < x ? y : x;
  }
  return x;
}

// Scalars and reduction scratch of a lane's epilogue (shared memory, 8-byte aligned base).
struct EpScratch {
  float* w;                  // [G][kMaxSplits] split weights of the output combination
  float* M;                  // [8] global max logit per query head
  float* linv;               // [8]
  float* Z;                  // [8]
  float* misc;               // [8] w_j, w_r
  int* i32;                  // [64] flags, j, r
  unsigned long long* u64;   // [128]: [0..63] sums, [64..95] minima and their slots, [96..103] Z partial per head, [104..105] pick key
  __host__ __device__ static constexpr int bytes(int G) { return (G * kMaxSplits + 32 + 64) * 4 + 128 * 8; }
  __device__ __forceinline__ void carve(unsigned char* base, int G) {
    w = reinterpret_cast<float*>(base);
    M = w + G * kMaxSplits;
    linv = M + 8;
    Z = linv + 8;
    misc = Z + 8;
    i32 = reinterpret_cast<int*>(misc + 8);
    u64 = reinterpret_cast<unsigned long long*>(i32 + 64);
  }
};

// ------------------------------------------------------------------------------------------------
// compile-time shape of one instantiation and its shared-memory carve-up
// ------------------------------------------------------------------------------------------------
template <typename T, int D, int G>
struct Cfg {
  static constexpr int kRowBytes = D * (int)sizeof(T);
  static constexpr int kTileBytes = kTileSlots * kRowBytes; // the K tile of a stage
  static constexpr int kLanesPerRow = G <= 2 ? 8 : 16;      // threads that share one cache row in the scan
  // Four query heads on bf16 rows: the P.V half of the scan (outside the reproducible chain) runs on mma.m16n8k8 with
  // the value fragments fetched by ldmatrix.trans.  The V tile of a stage is then written by tensor-map copies with the
  // 128-byte swizzle, one per 128-byte half of the rows ([half][32 rows][128 B], the 16-byte chunk index XORed with
  // row % 8), so that the eight rows of a fragment fall into eight different bank groups.
  static constexpr bool kMmaPV = G == 4 && sizeof(T) == 2 && D % 64 == 0;
  static constexpr int kVHalves = kRowBytes / 128;          // kMmaPV only
  static constexpr int kVHalfBytes = kTileSlots * 128;
  static constexpr int kStageBytes = 2 * kTileBytes;
  static constexpr int kFit = WKV_RING_BYTES / (2 * kTileBytes);
  static constexpr int kStages = kFit < 2 ? 2 : (kFit > 8 ? 8 : kFit);
  static constexpr int kRingBytes = kStages * kStageBytes;
  static constexpr int kAuxBytes = 2 * kRowBytes;           // k row and v row of the new token
  static constexpr int kWarpPartFloats = kConsumerWarps * G * (D + 2);
  static constexpr int kCtaPartFloats = G * (D + 2);
  // ring | new token rows | warp partials | mbarriers: all that a scan kernel uses
  static constexpr int kScanBytes = kRingBytes + kAuxBytes + kWarpPartFloats * 4 + 2 * kStages * 8 + 128;
  // ring | new token rows | warp partials | mbarriers | CTA partial | epilogue scalars | (cluster: chunk logits)
  static constexpr int kFixedBytes = kRingBytes + kAuxBytes + (kWarpPartFloats + kCtaPartFloats) * 4 + 2 * kStages * 8 +
                                     EpScratch::bytes(G) + 128;
};

template <typename T, int D, int G>
struct Smem {
  unsigned char* ring;       // [stage][K tile | V tile]
  T* aux;                    // [ k: D | v: D ] this step's token
  float* warp_part;          // [warp][G][D+2] : m, l, o[D]
  float* cta_part;           // [G][D+2]
  uint64_t* full_bar;        // [kStages]
  uint64_t* empty_bar;       // [kStages]
  EpScratch ep;              // epilogue scalars and reduction scratch
  float* chunk_logits;       // [G][chunk_cap] (cluster kernel only)
  __device__ __forceinline__ explicit Smem(unsigned char* raw) {
    using C = Cfg<T, D, G>;
    ring = raw;
    aux = reinterpret_cast<T*>(ring + C::kRingBytes);
    warp_part = reinterpret_cast<float*>(ring + C::kRingBytes + C::kAuxBytes);
    full_bar = reinterpret_cast<uint64_t*>(warp_part + C::kWarpPartFloats);
    empty_bar = full_bar + C::kStages;
    cta_part = reinterpret_cast<float*>(empty_bar + C::kStages);
    ep.carve(reinterpret_cast<unsigned char*>(cta_part + C::kCtaPartFloats), G);
    chunk_logits = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(cta_part + C::kCtaPartFloats) + EpScratch::bytes(G));
  }
  __device__ __forceinline__ T* aux_k(int) const { return aux; }
  __device__ __forceinline__ T* aux_v(int) const { return aux + D; }
};

// What the threads working on a unit know about its lane and its share of the lane's slots.
template <typename T>
struct LaneView {
  long long lane;            // global lane index
  int lane_local, b, hk, split;
  int len, t, new_slot, L;   // L = entries attended this step (new token included)
  int tile_begin, n_tiles;   // this unit's tiles
  int slot_begin, slot_end;  // this unit's slots [slot_begin, slot_end) clipped to L
  const T *Kl, *Vl;          // the lane's cache rows
  const T *new_k, *new_v;    // this step's token (shared memory)
  int* st;                   // the lane's state words
  int head, tail;            // chain ends before this step (only the code that finishes the lane reads them)
  int step;                  // set and used only by the kernel that finishes a whole block of a blocked prompt tail (kLoop):
  int row0;                  // the token's index inside its block, and the first row of its logits / probabilities
  int* st_s;                 // ... shared-memory copy of the state words, kept current from token to token
  const float* lgx_s;        // ... the lane's logits against the block's own keys [rows][block_tokens], in shared memory
};
// Index of the step's token inside its block, and first row of its logits / probabilities among the lane's rows: launch
// parameters, except in the kernel that loops over a block's tokens (kLoop), where they change from step to step.
template <bool kLoop, typename T>
__device__ __forceinline__ int step_of(const StepParams& P, const LaneView<T>& v) { return kLoop ? v.step : P.block_step; }
template <bool kLoop, typename T>
__device__ __forceinline__ int row0_of(const StepParams& P, const LaneView<T>& v) { return kLoop ? v.row0 : P.logit_row0; }

// Lane-level part of a view: addresses and the even deal of tiles (the first tiles_total % n_splits units get one more).
template <typename T, int D>
__device__ __forceinline__ void fill_view(LaneView<T>& v, const StepParams& P, int lane_local, int split, int len, int t,
                                          int new_slot) {
  v.lane_local = lane_local;
  v.split = split;
  v.b = lane_local / P.n_kv_heads;
  v.hk = lane_local % P.n_kv_heads;
  v.lane = (long long)P.lane0 + lane_local;
  v.st = P.lane_state + v.lane * LS_STRIDE;
  v.len = len;
  v.t = t;
  v.new_slot = new_slot;
  v.head = -1;
  v.tail = -1;
  v.L = len + 1;
  v.Kl = reinterpret_cast<const T*>(P.Kc) + v.lane * (long long)P.cap * D;
  v.Vl = reinterpret_cast<const T*>(P.Vc) + v.lane * (long long)P.cap * D;
  const int tiles_total = (v.L + kTileSlots - 1) / kTileSlots;
  const int base = tiles_total / P.n_splits, extra = tiles_total % P.n_splits;
  v.tile_begin = split * base + min(split, extra);
  v.n_tiles = base + (split < extra ? 1 : 0);
  v.slot_begin = min(v.L, v.tile_begin * kTileSlots);
  v.slot_end = min(v.L, (v.tile_begin + v.n_tiles) * kTileSlots);
}

// The flat deal of the two-kernel schedule.  The tiles of all lanes of a launch, P.tiles_cap per lane, form one
// sequence, lane after lane, and CTA i scans tiles [i*c, (i+1)*c) of it, c = P.flat_chunk: every CTA gets the same
// number of tiles whatever the number of lanes, so one wave of CTAs fills every SM equally -- with whole units per lane
// the CTA count is a multiple of the lane count and the SMs hold unequal numbers of them.  A CTA's range may end one
// lane and begin the next: per lane it holds a "piece", which it treats as the even deal treats a unit (own partial,
// own report to the lane's epilogue).  The pieces of a lane belong to consecutive CTAs.
// first CTA and number of pieces (units) of a lane, under either deal
__device__ __forceinline__ void lane_pieces(const StepParams& P, int lane_local, int& first_cta, int& n_pieces) {
  if (P.flat_chunk == 0) {
    first_cta = lane_local * P.n_splits;
    n_pieces = P.n_splits;
  } else {
    const long long g0 = (long long)lane_local * P.tiles_cap;
    first_cta = (int)(g0 / P.flat_chunk);
    n_pieces = (int)((g0 + P.tiles_cap - 1) / P.flat_chunk) - first_cta + 1;
  }
}
// The piece of lane `lane_local` that CTA `cta` holds under the flat deal: tiles [tb, te) of the lane, clipped to the
// tiles the lane really has; sets the view's share and returns the piece's index among the lane's pieces.
template <typename T>
__device__ __forceinline__ int flat_piece(LaneView<T>& v, const StepParams& P, int lane_local, int cta) {
  const long long lane_g0 = (long long)lane_local * P.tiles_cap;
  const long long g0 = (long long)cta * P.flat_chunk, g1 = g0 + P.flat_chunk;
  const int tb = (int)max(g0 - lane_g0, 0ll), te = (int)min(g1 - lane_g0, (long long)P.tiles_cap);
  const int tiles_total = (v.L + kTileSlots - 1) / kTileSlots;
  v.tile_begin = min(tb, tiles_total);
  v.n_tiles = max(0, min(te, tiles_total) - tb);
  v.slot_begin = min(v.L, tb * kTileSlots);
  v.slot_end = min(v.L, te * kTileSlots);
  v.split = cta - (int)(lane_g0 / P.flat_chunk);
  return v.split;
}

// Producer side of one ring stage (one thread): `rows` cache rows of K in one bulk copy and the same rows of V in one
// more -- or, where the stage keeps its V rows swizzled (Cfg::kMmaPV), whole 32-row boxes of V through the tensor map
// `vmap` over the value cache as a [rows_total][D] matrix, starting at row `vrow0` (rows past the lane's entries are
// other slots' bytes or, past the end of the cache, zero fill; the consumers never use them).
template <typename T, int D, int G>
__device__ __forceinline__ void fill_stage(unsigned char* dst, const T* Ksrc, const T* Vsrc, int rows, uint64_t* bar,
                                           const void* vmap, int vrow0) {
  using C = Cfg<T, D, G>;
  const uint32_t bytes = (uint32_t)rows * C::kRowBytes;
  // The cache rows are read once per step and there are far more of them than L2 holds; what the lane epilogues read
  // soon after (parked logits, split partials, scores and positions) should outlive them there: the tiles are marked to
  // leave L2 first (measured: 1.3 % of a step at 512 lanes x 4097 entries, 2.9 % with four query heads per key).
  const uint64_t pol = l2_policy_evict_first();
  if constexpr (!C::kMmaPV) {
    mbar_expect_tx(bar, 2 * bytes);
    bulk_g2s_hint(dst, Ksrc, bytes, bar, pol);
    bulk_g2s_hint(dst + C::kTileBytes, Vsrc, bytes, bar, pol);
  } else {
    mbar_expect_tx(bar, bytes + C::kVHalves * C::kVHalfBytes);
    bulk_g2s_hint(dst, Ksrc, bytes, bar, pol);
#pragma unroll
    for (int h = 0; h < C::kVHalves; ++h)
      tensor_g2s_2d_hint(dst + C::kTileBytes + h * C::kVHalfBytes, vmap, h * 64, vrow0, bar, pol);
  }
}

// ------------------------------------------------------------------------------------------------
// the scan: per-thread state of the four consumer warps (each warp owns 8 rows of every tile)
// ------------------------------------------------------------------------------------------------
// A row (one cache entry) is shared by LPR threads.  Thread l of the group owns the partial sums {l, l+LPR, ...} of
// the reproducible dot, each a block of D/16 contiguous channels, so butterfly rounds with off >= LPR are additions
// inside the thread and only log2(LPR) shuffles remain.
template <typename T, int D, int G>
struct Scanner {
  using C = Cfg<T, D, G>;
  static constexpr int LPR = C::kLanesPerRow;    // 8 or 16 threads per row
  static constexpr int NP = 16 / LPR;            // partial sums per thread
  static constexpr int CH = D / 16;              // channels per partial sum
  static constexpr int CP = CH / 2;              // ... as (even, odd) channel pairs: the arithmetic is packed fp32x2
  static constexpr int RPP = 32 / LPR;           // rows per warp pass
  static constexpr int PASSES = 8 / RPP;
  // With G query heads the butterfly is run as a reduce-scatter: each round with more than one head left halves the
  // heads a thread carries, so a row's LPR threads end up owning one head each (LH threads per head) and the softmax
  // bookkeeping is done once per head instead of once per thread.  The additions are those of the plain butterfly.
  static constexpr int LH = LPR / G;             // threads per (row, head) after the reduce-scatter
  static_assert(G <= LPR && LH >= 1, "at most one head per thread of a row");
  // P.V on the tensor cores (C::kMmaPV): per warp and tile, (V rows)^T [channels x 8 rows] times the probabilities
  // [8 rows x (4 heads as bf16 high parts | 4 heads as bf16 low parts)], in blocks of 16 channels.  Lane t = 4*c + q holds
  // channels 16*blk + c and 16*blk + 8 + c of columns 2q and 2q+1; end() adds the low-part columns to the high-part ones.
  static constexpr bool MMA = C::kMmaPV;
  static constexpr int NB = D / 16;              // channel blocks
  f32x2 qf[G][NP][CP];
  float m_run, l_run;                            // online softmax of this thread's head: head_of(l) = l / LH
  f32x2 o_acc[MMA ? 1 : G][NP][CP];
  float oc[MMA ? NB : 1][4];

  __device__ __forceinline__ void begin(const T* q) {      // q: [G][D], 16-byte aligned (global or shared)
    const int l = (threadIdx.x & 31) % LPR;
    m_run = -INFINITY;
    l_run = 0.f;
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
      for (int j = 0; j < NP; ++j) load_pairs<CP>(q + g * D + (l + LPR * j) * CH, qf[g][j]);
      if constexpr (!MMA) {
#pragma unroll
        for (int j = 0; j < NP; ++j)
#pragma unroll
          for (int e = 0; e < CP; ++e) o_acc[g][j][e] = 0ull;
      }
    }
    if constexpr (MMA) {
#pragma unroll
      for (int j = 0; j < NB; ++j) oc[j][0] = oc[j][1] = oc[j][2] = oc[j][3] = 0.f;
    }
  }
  // The same start for query rows that are not contiguous: row r is head r % group of token min(r / group, n_tok - 1),
  // tokens tok_stride elements apart (the blocked prompt tail scans for several tokens of a prompt at once).
  __device__ __forceinline__ void begin_rows(const T* q, long long tok_stride, int group, int n_tok) {
    const int l = (threadIdx.x & 31) % LPR;
    m_run = -INFINITY;
    l_run = 0.f;
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const T* row = q + (long long)min(g / group, n_tok - 1) * tok_stride + (long long)(g % group) * D;
#pragma unroll
      for (int j = 0; j < NP; ++j) load_pairs<CP>(row + (l + LPR * j) * CH, qf[g][j]);
    }
  }
  // 32-bit word w of row `row` of a stage's V tile: plain rows, or (MMA) the swizzled halves that the tensor-map copies
  // leave -- [half][row][128 B] with address bits 4..6 XORed with bits 7..9 (the tile starts on a 1024-byte boundary).
  __device__ __forceinline__ static uint32_t* v_word(T* tV, int row, int w) {
    if constexpr (!MMA) return reinterpret_cast<uint32_t*>(tV + row * D) + w;
    unsigned char* base = reinterpret_cast<unsigned char*>(tV);
    const int chunk = w >> 2;                                           // 16-byte chunk of the row
    return reinterpret_cast<uint32_t*>(base + (chunk >> 3) * C::kVHalfBytes + row * 128 + ((((chunk & 7) ^ (row & 7)) << 4) | ((w & 3) << 2)));
  }

  // value of head g's owner threads, for every thread of the row group
  __device__ __forceinline__ static float from_head(float mine, int g) {
    if constexpr (G == 1) return mine;
    const int lane_id = threadIdx.x & 31;
    return __shfl_sync(0xffffffffu, mine, (lane_id & ~(LPR - 1)) | (g * LH));
  }

  // Tensor-core P.V of one tile (MMA configurations): oc += (the warp's 8 value rows)^T . (their probabilities).
  // `mine` is the probability of this thread's own (row, head): row 2*li + rg of the warp's eight, head my_head.
  __device__ __forceinline__ void pv_mma(T* tV, float mine, int slot0, int L) {
    const int warp = threadIdx.x >> 5, lane_id = threadIdx.x & 31;
    if (slot0 + kTileSlots > L) {
      // ragged tile: rows beyond L hold stale bytes, possibly NaN patterns, and 0 * NaN would reach the accumulators
      for (int w = lane_id; w < 8 * (C::kRowBytes / 4); w += 32) {
        const int r = w / (C::kRowBytes / 4);
        if (slot0 + warp * 8 + r >= L) *v_word(tV, warp * 8 + r, w % (C::kRowBytes / 4)) = 0u;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
    }
    // B fragment: lane t = 4*n + q supplies rows 2q, 2q+1 of column n (n < 4: head n, high part; else head n-4, low
    // part).  Row 2q is pass q of row group 0, row 2q+1 pass q of row group 1; head n % 4 is this lane's own head.
    const float other = __shfl_xor_sync(0xffffffffu, mine, 16);
    const bool up = lane_id >= 16;
    const float pe = up ? other : mine, po = up ? mine : other;
    const __nv_bfloat16 he = __float2bfloat16_rn(pe), ho = __float2bfloat16_rn(po);
    const __nv_bfloat16 le = __float2bfloat16_rn(pe - __bfloat162float(he)), lo = __float2bfloat16_rn(po - __bfloat162float(ho));
    const uint32_t b0 = up ? (bf16_bits(le) | (bf16_bits(lo) << 16)) : (bf16_bits(he) | (bf16_bits(ho) << 16));
    // lanes 8i..8i+7 address rows 0..7 of the warp's share, 16-byte chunk 4*jj + i of the row (channels 32*jj + 8*i ...)
#pragma unroll
    for (int jj = 0; jj < NB / 2; ++jj) {
      uint32_t af[4];
      ldmatrix_x4_trans(af, v_word(tV, warp * 8 + (lane_id & 7), (4 * jj + (lane_id >> 3)) * 4));
      mma_m16n8k8_bf16(oc[2 * jj], af[0], af[1], b0);
      mma_m16n8k8_bf16(oc[2 * jj + 1], af[2], af[3], b0);
    }
  }

  // The cache copy of this step's token may still be in flight: the warp that owns its row overwrites the row in the
  // tile (the K tile, the V tile or both: a null pointer skips one) with the token's k and v before anybody reads it.
  __device__ __forceinline__ static void patch_new_token(T* tK, T* tV, int slot0, int new_slot, const T* new_k, const T* new_v) {
    const int warp = threadIdx.x >> 5, lane_id = threadIdx.x & 31;
    const int ns_row = new_slot - slot0;
    if (ns_row >= warp * 8 && ns_row < warp * 8 + 8) {
      const uint32_t* sk = reinterpret_cast<const uint32_t*>(new_k);
      const uint32_t* sv_ = reinterpret_cast<const uint32_t*>(new_v);
      for (int w = lane_id; w < C::kRowBytes / 4; w += 32) {
        if (tK != nullptr) reinterpret_cast<uint32_t*>(tK + ns_row * D)[w] = sk[w];
        if (tV != nullptr) *v_word(tV, ns_row, w) = sv_[w];
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // before the stage is refilled by a bulk copy
      __syncwarp();
    }
  }

  // Logits of my head for the rows of my row group, one per pass (the reproducible dot; -inf for rows beyond L).
  __device__ __forceinline__ void logits(const T* tK, int slot0, int L, float scale, float (&sv)[PASSES], bool (&valid)[PASSES]) const {
    const int warp = threadIdx.x >> 5, lane_id = threadIdx.x & 31;
    const int rg = lane_id / LPR, l = lane_id % LPR;
#pragma unroll
    for (int ps = 0; ps < PASSES; ++ps) {
      const int row = warp * 8 + ps * RPP + rg;
      valid[ps] = slot0 + row < L;
      f32x2 kf[NP][CP];
#pragma unroll
      for (int j = 0; j < NP; ++j) load_pairs<CP>(tK + row * D + (l + LPR * j) * CH, kf[j]);
      float vals[G];
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float pp[NP];
#pragma unroll
        for (int j = 0; j < NP; ++j) {
          f32x2 acc = 0ull;                                            // (even-channel chain, odd-channel chain)
#pragma unroll
          for (int e = 0; e < CP; ++e) acc = fma2(qf[g][j][e], kf[j][e], acc);
          pp[j] = __fadd_rn(lo_of(acc), hi_of(acc));
        }
        vals[g] = pp[0];
        if constexpr (NP == 2) vals[g] = __fadd_rn(pp[0], pp[1]);      // butterfly round off = 8
      }
      // butterfly rounds off = LPR/2 .. 1: p_r + p_{r^off}; while several heads are left, each partner keeps half
#pragma unroll
      for (int off = LPR / 2, n = G; off >= 1; off >>= 1) {
        if (n > 1) {
          const bool upper = (l & off) != 0;
#pragma unroll
          for (int i = 0; i < n / 2; ++i) {
            const float keep = upper ? vals[n / 2 + i] : vals[i];
            const float send = upper ? vals[i] : vals[n / 2 + i];
            vals[i] = __fadd_rn(keep, __shfl_xor_sync(0xffffffffu, send, off));
          }
          n >>= 1;
        } else {
          vals[0] = __fadd_rn(vals[0], __shfl_xor_sync(0xffffffffu, vals[0], off));
        }
      }
      const float sc = __fmul_rn(scale, vals[0]);
      sv[ps] = valid[ps] ? sc : -INFINITY;
    }
  }

  // Park the logits of my head at logit_dst[head * logit_stride + slot - logit_off]: thread li of the head's LH threads
  // takes the passes ps with ps % LH == li.
  __device__ __forceinline__ static void park(const float (&sv)[PASSES], int slot0, int L, float* logit_dst,
                                              long long logit_stride, int logit_off) {
    const int warp = threadIdx.x >> 5, lane_id = threadIdx.x & 31;
    const int rg = lane_id / LPR, l = lane_id % LPR;
    const int my_head = l / LH, li = l % LH;
#pragma unroll
    for (int ps = 0; ps < PASSES; ++ps) {
      const int slot = slot0 + warp * 8 + ps * RPP + rg;
      if ((ps % LH) == li && slot < L) logit_dst[(long long)my_head * logit_stride + (slot - logit_off)] = sv[ps];
    }
  }

  // One tile of up to 32 rows starting at slot0; logits parked at logit_dst[g*logit_stride + slot - logit_off].
  __device__ __forceinline__ void tile(T* tK, T* tV, int slot0, int L, int new_slot, const T* new_k, const T* new_v,
                                       float scale, float* logit_dst, long long logit_stride, int logit_off) {
    const float kLog2e = 1.4426950408889634f;
    const int warp = threadIdx.x >> 5, lane_id = threadIdx.x & 31;
    const int rg = lane_id / LPR, l = lane_id % LPR;
    const int li = l % LH;
    patch_new_token(tK, tV, slot0, new_slot, new_k, new_v);
    float sv[PASSES];                                                // logits of my head, one row per pass
    bool valid[PASSES];
    logits(tK, slot0, L, scale, sv, valid);
    park(sv, slot0, L, logit_dst, logit_stride, logit_off);
    // online softmax update of my head, one rescale per tile
    float corr;
    {
      float mt = sv[0];
#pragma unroll
      for (int ps = 1; ps < PASSES; ++ps) mt = fmaxf(mt, sv[ps]);
      if constexpr (MMA) mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 16));   // one accumulator for the warp's 8 rows
      const float m_new = fmaxf(m_run, mt);
      const float m_use = m_new == -INFINITY ? 0.f : m_new;
      corr = fast_exp2((m_run - m_use) * kLog2e);
      m_run = m_new;
      l_run *= corr;
#pragma unroll
      for (int ps = 0; ps < PASSES; ++ps) {
        sv[ps] = fast_exp2((sv[ps] - m_use) * kLog2e);                 // now probabilities (0 for rows beyond L)
        l_run += sv[ps];
      }
    }
    if constexpr (MMA) {
      static_assert(PASSES == 4 && LH == 4 && RPP == 2, "fragment layout below assumes 16 threads per row, 4 heads");
      if (__any_sync(0xffffffffu, corr != 1.0f)) {
        const int src = (lane_id & 1) * 8;                             // my columns' heads: 2*(q & 1) and the next one
        const float ca = __shfl_sync(0xffffffffu, corr, src), cb = __shfl_sync(0xffffffffu, corr, src + LH);
#pragma unroll
        for (int j = 0; j < NB; ++j) { oc[j][0] *= ca; oc[j][1] *= cb; oc[j][2] *= ca; oc[j][3] *= cb; }
      }
      const float mine = li == 0 ? sv[0] : (li == 1 ? sv[1] : (li == 2 ? sv[2] : sv[3]));
      pv_mma(tV, mine, slot0, L);
    } else {
    // the running maxima settle after a few tiles: rescale the output accumulators only when some head's maximum moved
    if (__any_sync(0xffffffffu, corr != 1.0f)) {
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float cg = from_head(corr, g);
        const f32x2 corr2 = pack2(cg, cg);
#pragma unroll
        for (int j = 0; j < NP; ++j)
#pragma unroll
          for (int e = 0; e < CP; ++e) o_acc[g][j][e] = mul2(o_acc[g][j][e], corr2);
      }
    }
#pragma unroll
    for (int ps = 0; ps < PASSES; ++ps) {
      const int row = warp * 8 + ps * RPP + rg;
      f32x2 vf[NP][CP];
#pragma unroll
      for (int j = 0; j < NP; ++j) load_pairs<CP>(tV + row * D + (l + LPR * j) * CH, vf[j]);
      float pg[G];
#pragma unroll
      for (int g = 0; g < G; ++g) pg[g] = from_head(sv[ps], g);
      if (valid[ps]) {                                                 // rows beyond L hold stale bytes, possibly NaN
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const f32x2 p2 = pack2(pg[g], pg[g]);
#pragma unroll
          for (int j = 0; j < NP; ++j)
#pragma unroll
            for (int e = 0; e < CP; ++e) o_acc[g][j][e] = fma2(p2, vf[j][e], o_acc[g][j][e]);
        }
      }
    }
    }  // !MMA
  }

  // Fold the warp's row groups and leave the warp's partial (m, l, o[D]) per query head in shared memory.
  __device__ __forceinline__ void end(float* warp_part) {
    const float kLog2e = 1.4426950408889634f;
    const int warp = threadIdx.x >> 5, lane_id = threadIdx.x & 31;
    const int rg = lane_id / LPR, l = lane_id % LPR;
    const int my_head = l / LH, li = l % LH;
    if constexpr (MMA) {
      l_run += __shfl_xor_sync(0xffffffffu, l_run, 16);               // both row groups ran on the same maximum
      const int c = lane_id >> 2, q = lane_id & 3;
#pragma unroll
      for (int j = 0; j < NB; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) oc[j][i] += __shfl_xor_sync(0xffffffffu, oc[j][i], 2);   // high-part + low-part columns
      if (q < 2) {
        float* wa = warp_part + (warp * G + 2 * q) * (D + 2) + 2;
        float* wb = wa + (D + 2);
#pragma unroll
        for (int j = 0; j < NB; ++j) {
          wa[16 * j + c] = oc[j][0];
          wb[16 * j + c] = oc[j][1];
          wa[16 * j + 8 + c] = oc[j][2];
          wb[16 * j + 8 + c] = oc[j][3];
        }
      }
      if (rg == 0 && li == 0) {
        float* wp = warp_part + (warp * G + my_head) * (D + 2);
        wp[0] = m_run;
        wp[1] = l_run;
      }
    } else {
#pragma unroll
    for (int off = 16; off >= LPR; off >>= 1) {
      const float m_o = __shfl_xor_sync(0xffffffffu, m_run, off);     // same head on both sides
      const float l_o = __shfl_xor_sync(0xffffffffu, l_run, off);
      const float m_new = fmaxf(m_run, m_o);
      const float m_use = m_new == -INFINITY ? 0.f : m_new;
      const float c_me = fast_exp2((m_run - m_use) * kLog2e), c_o = fast_exp2((m_o - m_use) * kLog2e);
      l_run = l_run * c_me + l_o * c_o;
      m_run = m_new;
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float cm = from_head(c_me, g), co = from_head(c_o, g);
        const f32x2 c_me2 = pack2(cm, cm), c_o2 = pack2(co, co);
#pragma unroll
        for (int j = 0; j < NP; ++j)
#pragma unroll
          for (int e = 0; e < CP; ++e) {
            const f32x2 o_o = __shfl_xor_sync(0xffffffffu, o_acc[g][j][e], off);
            o_acc[g][j][e] = fma2(o_acc[g][j][e], c_me2, mul2(o_o, c_o2));
          }
      }
    }
    if (rg == 0) {
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float* wp = warp_part + (warp * G + g) * (D + 2);
#pragma unroll
        for (int j = 0; j < NP; ++j)
#pragma unroll
          for (int e = 0; e < CP; ++e) {
            wp[2 + (l + LPR * j) * CH + 2 * e] = lo_of(o_acc[g][j][e]);
            wp[2 + (l + LPR * j) * CH + 2 * e + 1] = hi_of(o_acc[g][j][e]);
          }
      }
      if (li == 0) {
        float* wp = warp_part + (warp * G + my_head) * (D + 2);
        wp[0] = m_run;
        wp[1] = l_run;
      }
    }
    }  // !MMA
  }
};

// The four warp partials -> one (m, l, o[D]) per query head at dst (shared or global).  Call after the group's barrier.
template <int D, int G, int NT>
__device__ __forceinline__ void combine_warps(const float* warp_part, float* dst) {
  const float kLog2e = 1.4426950408889634f;
  for (int idx = threadIdx.x; idx < G * D; idx += NT) {
    const int g = idx / D, c = idx % D;
    float mx = -INFINITY;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; ++w) mx = fmaxf(mx, warp_part[(w * G + g) * (D + 2)]);
    const float m_use = mx == -INFINITY ? 0.f : mx;
    float o = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; ++w) {
      const float* wp = warp_part + (w * G + g) * (D + 2);
      const float cw = fast_exp2((wp[0] - m_use) * kLog2e);
      o += wp[2 + c] * cw;
      l += wp[1] * cw;
    }
    dst[g * (D + 2) + 2 + c] = o;
    if (c == 0) { dst[g * (D + 2)] = mx; dst[g * (D + 2) + 1] = l; }
  }
}

// ------------------------------------------------------------------------------------------------
// epilogue pieces (reproducible arithmetic), run by the first NT threads of a CTA
// ------------------------------------------------------------------------------------------------
// e_i = exp(s_i - M_g), written back in place of the logit, and this thread's share of sum_i trunc(e_i * 2^40).
// Element i of the range lives at lg[g*stride + i]; kL2 selects loads that bypass L1 (logits written by other SMs).
template <int G, bool kL2, int NT>
__device__ __forceinline__ void exp_and_zsum(float* lg, long long stride, int n, const float* M, unsigned long long (&zl)[G]) {
  constexpr int U = 4;                          // loads of U elements are issued before any of them is used
#pragma unroll
  for (int g = 0; g < G; ++g) zl[g] = 0ull;
  for (int i0 = threadIdx.x; i0 < n; i0 += NT * U) {
    float sx[G][U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * NT;
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float* p = lg + (long long)g * stride + i;
        sx[g][u] = i < n ? (kL2 ? __ldcg(p) : *p) : 0.f;
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * NT;
      if (i < n) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const float e = repro_exp(__fsub_rn(sx[g][u], M[g]));
          lg[(long long)g * stride + i] = e;    // re-read by the same thread in fold_scores
          zl[g] += __float2ull_rz(__fmul_rn(e, 1099511627776.0f));
        }
      }
    }
  }
}

// Group-wide sums of G 64-bit integers; x[g] holds the total in every thread after the call.  scratch: G*NT/32 entries.
// kRelease = false leaves out the trailing barrier: the caller then must not write the scratch again before a later
// barrier of its own.
template <int G, int NT, bool kRelease = true>
__device__ __forceinline__ void group_sum_u64(unsigned long long (&x)[G], unsigned long long* scratch) {
  const int warp = threadIdx.x >> 5, lane_id = threadIdx.x & 31;
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const unsigned long long w = warp_sum_u64(x[g]);
    if (lane_id == 0) scratch[g * (NT / 32) + warp] = w;
  }
  group_sync<NT>();
#pragma unroll
  for (int g = 0; g < G; ++g) {
    unsigned long long z = 0ull;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) z += scratch[g * (NT / 32) + w];
    x[g] = z;
  }
  if constexpr (kRelease) group_sync<NT>();
}

// One slot's share of a step: p = e / Z per query head (written to the optional probability output), the group mean
// folded into the slot's accumulated score (Algorithm 1: a = [a,0] + A_t), abar = a / n and the pick key.
template <typename T, int G, bool kLoop = false>
__device__ __forceinline__ void fold_one(const StepParams& P, const LaneView<T>& v, float* a_l, int32_t* pos_l, int slot,
                                         const float (&e)[G], const float* Z, float a_old, int pos_i, bool compress,
                                         unsigned long long& best, int& best_slot, float* a_s = nullptr) {
  float pg[G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    pg[g] = __fdiv_rn(e[g], Z[g]);
    if (P.probs) P.probs[((long long)v.lane_local * P.probs_rows + row0_of<kLoop>(P, v) + g) * P.probs_stride + slot] = pg[g];
  }
  float pbar = pg[0];
#pragma unroll
  for (int g = 1; g < G; ++g) pbar = __fadd_rn(pbar, pg[g]);
  if (G > 1) pbar = __fmul_rn(pbar, 1.0f / (float)G);
  const float a_new = __fadd_rn(a_old, pbar);
  a_l[slot] = a_new;
  if constexpr (kLoop) a_s[slot] = a_new;              // the staged copy serves the block's next token (and the merge weights)
  if (slot == v.new_slot) pos_l[slot] = v.t;
  if (compress && pos_i >= P.sink && pos_i <= v.t - P.window) {
    const float abar = __fdiv_rn(a_new, __int2float_rn(v.t - pos_i + 1));
    const unsigned long long key = ((unsigned long long)__float_as_uint(abar) << 32) | (uint32_t)pos_i;
    if (key < best) { best = key; best_slot = slot; }
  }
}

// A_t over a range of slots, a = [a,0] + A_t, abar = a/n and the range's pick key (Algorithm 1).
// e values at lg[g*stride + i] for slot slot0 + i.  Updates the thread's best (key, slot).
template <typename T, int G, int NT>
__device__ __forceinline__ void fold_scores(const StepParams& P, const LaneView<T>& v, const float* lg, long long stride,
                                            int slot0, int n, const float* Z, bool compress, unsigned long long& best,
                                            int& best_slot) {
  float* a_l = P.a + v.lane * P.cap;
  int32_t* pos_l = P.pos + v.lane * P.cap;
  const int t = v.t;
  constexpr int U = 4;                          // a, pos and e of U slots are loaded before any of them is used
  for (int i0 = threadIdx.x; i0 < n; i0 += NT * U) {
    float a_old[U], ev[U][G];
    int pos_v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * NT;
      const int slot = slot0 + i;
      const bool ok = i < n, is_new = slot == v.new_slot;
      a_old[u] = (ok && !is_new) ? a_l[slot] : 0.f;
      pos_v[u] = (ok && !is_new) ? pos_l[slot] : t;
#pragma unroll
      for (int g = 0; g < G; ++g) ev[u][g] = ok ? lg[(long long)g * stride + i] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * NT;
      if (i >= n) continue;
      fold_one<T, G>(P, v, a_l, pos_l, slot0 + i, ev[u], Z, a_old[u], pos_v[u], compress, best, best_slot);
    }
  }
}

// Group-wide minimum of the pick key and the slot that owns it, in every thread (slot_out: -1 when no slot is
// evictable).  scratch: NT/32 keys followed by NT/32 slot words (as 64-bit entries); one barrier, after which the
// caller must not write the scratch before a barrier of its own.
template <int NT>
__device__ __forceinline__ unsigned long long group_min_key(unsigned long long best, int best_slot, unsigned long long* scratch,
                                                            int& slot_out) {
  constexpr int NW = NT / 32;
  const int warp = threadIdx.x >> 5;
  const unsigned long long wmin = warp_min_u64(best);
  // positions are unique, so a key below ~0 has exactly one owner in the warp; ~0 means "no candidate" in every lane
  if (best == wmin && (best_slot >= 0 || (threadIdx.x & 31) == 0)) {
    scratch[warp] = wmin;
    scratch[NW + warp] = (unsigned long long)(long long)best_slot;
  }
  group_sync<NT>();
  unsigned long long bmin = scratch[0];
  int bslot = (int)(long long)scratch[NW];
#pragma unroll
  for (int w = 1; w < NW; ++w) {
    const unsigned long long k = scratch[w];
    if (k < bmin) { bmin = k; bslot = (int)(long long)scratch[NW + w]; }
  }
  slot_out = bslot;
  return bmin;
}

// Link the new entry as the chain's tail, unlink the victim j (Algorithm 1: remove K[j], a[j], n[j]; the right
// neighbour keeps its own key, a and n), merge V[j] into V[next[j]], update the lane state.  One group per lane runs it.
template <typename T, int D, int G, int NT, bool kLoop = false>
__device__ __forceinline__ void finish_lane(const StepParams& P, const LaneView<T>& v, const EpScratch& ep, bool compress,
                                            unsigned long long bmin, int j_slot, const float* a_s = nullptr,
                                            const int* pos_s = nullptr) {
  static_assert(NT >= D, "one thread per channel of the merged row");
  const int tid = threadIdx.x;
  const int t = v.t, new_slot = v.new_slot, L = v.L;
  float* a_l = P.a + v.lane * P.cap;
  int32_t* pos_l = P.pos + v.lane * P.cap;
  int32_t* next_l = P.next + v.lane * P.cap;
  int32_t* prev_l = P.prev + v.lane * P.cap;
  T* Vw = const_cast<T*>(v.Vl);
  // the victim's value row does not depend on the chain walk below: fetch it meanwhile
  // (the row of this step's token may have been written to the cache by other threads: v.new_v is the safe copy)
  float vj = 0.f;
  const bool merging = compress && P.merge && j_slot >= 0;
  const bool blocked = P.block_tokens > 0;               // blocked prompt tail: rows that this step changes are recorded
  if ((merging || (blocked && compress && j_slot >= 0)) && tid < D)
    vj = to_f32(j_slot == new_slot ? v.new_v[tid] : __ldcg(Vw + (long long)j_slot * D + tid));
  // ... and so can the right neighbour's row, without waiting for thread 0's walk: r = next[j], which this step
  // changes only if j is the old tail (then r is the new entry).  One round trip less on the lane's critical path.
  int r_early = -1;
  float vr_early = 0.f;
  if (merging && tid < D) {
    r_early = j_slot == v.tail ? new_slot : __ldcg(next_l + j_slot);
    if (r_early >= 0 && r_early < P.cap)
      vr_early = to_f32(r_early == new_slot ? v.new_v[tid] : __ldcg(Vw + (long long)r_early * D + tid));
  }
  if (tid == 0) {
    int head = v.head, tail = v.tail;
    next_l[new_slot] = -1;
    prev_l[new_slot] = tail;
    if (tail >= 0) next_l[tail] = new_slot; else head = new_slot;
    tail = new_slot;
    int ev_pos = -1, new_len = L, new_free = L;          // while growing, slots fill in arrival order
    ep.i32[2] = -1;
    if (compress) {
      const int j = j_slot;
      const int r = j >= 0 ? next_l[j] : -1;
      if (j < 0 || r < 0 || r >= P.cap) {
        atomicOr(P.status, kStatusBadLink);              // cannot happen with budget >= sink + window
      } else {
        const int pv = prev_l[j];
        const float abar_j = __uint_as_float((uint32_t)(bmin >> 32));
        // (kLoop: the staged copies are current -- this step's fold wrote them before the pick's barrier)
        const int pos_r = kLoop ? pos_s[r] : (r == new_slot ? t : __ldcg(pos_l + r));
        const float abar_r = __fdiv_rn(kLoop ? a_s[r] : __ldcg(a_l + r), __int2float_rn(t - pos_r + 1));
        const float Dn = __fadd_rn(abar_j, abar_r);
        float wj = 0.5f, wr = 0.5f;
        if (Dn != 0.f) { wj = __fdiv_rn(abar_j, Dn); wr = __fdiv_rn(abar_r, Dn); }
        ep.misc[0] = wj;
        ep.misc[1] = wr;
        ep.i32[2] = j;
        ep.i32[3] = r;
        ev_pos = (int)(uint32_t)(bmin & 0xffffffffull);
        if (pv >= 0) next_l[pv] = r; else head = r;
        prev_l[r] = pv;
        pos_l[j] = -1;
        new_len = P.budget;
        new_free = j;
      }
    }
    v.st[LS_LEN] = new_len;
    v.st[LS_T] = t + 1;
    v.st[LS_HEAD] = head;
    v.st[LS_TAIL] = tail;
    v.st[LS_FREE] = new_free;
    if constexpr (kLoop) {
      v.st_s[LS_LEN] = new_len;
      v.st_s[LS_T] = t + 1;
      v.st_s[LS_HEAD] = head;
      v.st_s[LS_TAIL] = tail;
      v.st_s[LS_FREE] = new_free;
    }
    if (P.evicted) P.evicted[v.b * P.ev_bs + v.hk + (kLoop ? (long long)v.step * P.ev_ts : 0ll)] = ev_pos;
    if (blocked) {
      int32_t* rs = P.rec_slot + ((long long)v.lane_local * P.block_tokens + step_of<kLoop>(P, v)) * 2;
      rs[0] = ep.i32[2];                                   // the removed entry's slot (-1: nothing removed)
      rs[1] = (ep.i32[2] >= 0 && P.merge) ? ep.i32[3] : -1;
    }
  }
  group_sync<NT>();
  // V[r] <- (abar_j V[j] + abar_r V[r]) / (abar_j + abar_r), stored in T
  if (merging && ep.i32[2] >= 0 && tid < D) {
    const int r = ep.i32[3];
    const float wj = ep.misc[0], wr = ep.misc[1];
    const float vr = r == r_early ? vr_early : to_f32(r == new_slot ? v.new_v[tid] : __ldcg(Vw + (long long)r * D + tid));
    Vw[(long long)r * D + tid] = from_f32<T>(__fmaf_rn(wj, vj, __fmul_rn(wr, vr)));
    if (blocked) P.rec_rows[(((long long)v.lane_local * P.block_tokens + step_of<kLoop>(P, v)) * 2 + 1) * D + tid] = vr;
  }
  if (blocked && compress && ep.i32[2] >= 0 && tid < D)
    P.rec_rows[(((long long)v.lane_local * P.block_tokens + step_of<kLoop>(P, v)) * 2) * D + tid] = vj;
}

// Steps (1) and (2) of a lane's epilogue from global scratch: the split weights, the global maximum and normaliser of
// every query head (left in ep.M / ep.linv / ep.w behind a barrier), and o_t.
template <typename T, int D, int G, int NT>
__device__ __forceinline__ void combine_partials(const StepParams& P, const LaneView<T>& v, const EpScratch& ep) {
  const float kLog2e = 1.4426950408889634f;
  const int tid = threadIdx.x;
  const float* part = P.part + (long long)v.lane_local * P.n_splits * G * (D + 2);
  int first_cta, n_pieces;
  lane_pieces(P, v.lane_local, first_cta, n_pieces);
  // (1) split weights and the global max / normaliser of every query head
  // (warp g takes head g, a lane takes splits lane and lane + 32: one round of loads instead of a serial loop)
  static_assert(NT / 32 >= G && kMaxSplits <= 64, "one warp per query head, two splits per lane");
  if ((tid >> 5) < G) {
    const int g = tid >> 5, lq = tid & 31;
    const float* pg = part + g * (D + 2);
    const long long st = (long long)G * (D + 2);
    const bool has0 = lq < n_pieces, has1 = lq + 32 < n_pieces;
    const float m0 = has0 ? __ldcg(pg + lq * st) : -INFINITY, l0 = has0 ? __ldcg(pg + lq * st + 1) : 0.f;
    const float m1 = has1 ? __ldcg(pg + (lq + 32) * st) : -INFINITY, l1 = has1 ? __ldcg(pg + (lq + 32) * st + 1) : 0.f;
    float M = fmaxf(m0, m1);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
    const float w0 = has0 ? fast_exp2((m0 - M) * kLog2e) : 0.f, w1 = has1 ? fast_exp2((m1 - M) * kLog2e) : 0.f;
    if (has0) ep.w[g * kMaxSplits + lq] = w0;
    if (has1) ep.w[g * kMaxSplits + lq + 32] = w1;
    float lsum = w0 * l0 + w1 * l1;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, off);
    if (lq == 0) {
      ep.M[g] = M;                  // max of the reproducible logits: exact, order-free
      ep.linv[g] = 1.f / lsum;
    }
  }
  group_sync<NT>();
  // (2) o_t = A_t^T V_t (Background section), V as it was before this step's merge
  {
    T* out = reinterpret_cast<T*>(P.out) + v.b * P.out_bs + (long long)v.hk * G * D;
    for (int idx = tid; idx < G * D; idx += NT) {
      const int g = idx / D, c = idx % D;
      const float* pg = part + g * (D + 2) + 2 + c;
      float o = 0.f;
      for (int s = 0; s < n_pieces; ++s) o += ep.w[g * kMaxSplits + s] * __ldcg(pg + (long long)s * G * (D + 2));
      out[idx] = from_f32<T>(o * ep.linv[g]);
    }
  }
}

// Zeroes of the optional probability output beyond the lane's entries.
template <int G, int NT>
__device__ __forceinline__ void clear_probs_tail(const StepParams& P, int lane_local, int row0, int L) {
  if (P.probs) {
    for (int i = L + (int)threadIdx.x; i < P.budget + 1; i += NT)
#pragma unroll
      for (int g = 0; g < G; ++g) P.probs[((long long)lane_local * P.probs_rows + row0 + g) * P.probs_stride + i] = 0.f;
  }
}

// The whole epilogue of a lane from global scratch (all partials and logits of the lane are visible to the caller).
template <typename T, int D, int G, int NT>
__device__ __forceinline__ void lane_epilogue_from_scratch(const StepParams& P, const LaneView<T>& v, const EpScratch& ep) {
  const int L = v.L;
  constexpr bool kLoop = false;
  float* lg = P.logits + ((long long)v.lane_local * P.logit_rows + P.logit_row0) * P.cap;
  combine_partials<T, D, G, NT>(P, v, ep);
  // (3) Z_g as an exact integer sum
  float Zr[G];
  {
    unsigned long long zl[G];
    exp_and_zsum<G, true, NT>(lg, P.cap, L, ep.M, zl);
    group_sum_u64<G, NT, false>(zl, ep.u64);          // every thread holds the totals; the scratch is not written again
#pragma unroll
    for (int g = 0; g < G; ++g) Zr[g] = __fmul_rn(__ull2float_rn(zl[g]), 1.0f / 1099511627776.0f);
  }
  // (4) probabilities, score fold, pick
  const bool compress = L > P.budget;                 // Algorithm 1's trigger: the list is longer than m
  unsigned long long best = ~0ull;
  int best_slot = -1;
  fold_scores<T, G, NT>(P, v, lg, P.cap, 0, L, Zr, compress, best, best_slot);
  clear_probs_tail<G, NT>(P, v.lane_local, row0_of<kLoop>(P, v), L);
  int j_slot;
  const unsigned long long bmin = group_min_key<NT>(best, best_slot, ep.u64 + 64, j_slot);   // its barrier also publishes a, pos
  // (5), (6)
  finish_lane<T, D, G, NT>(P, v, ep, compress, bmin, j_slot);
}

// The same epilogue for a lane of at most E * NT entries, with what a thread needs close at hand: thread tid owns slots
// tid, tid + NT, ...; their accumulated scores and positions are in shared memory (a_s, pos_s: staged by the caller
// before the lane's scan was even finished -- the scan writes neither; a thread reads back only what it staged itself)
// and their parked logits are requested here in one go and stay in registers, so the lane pays one round trip to L2
// where the loop version pays one per few slots and phase.  Same arithmetic, same results.
template <typename T, int D, int G, int NT, int E, bool kLoop = false>
__device__ __forceinline__ void lane_epilogue_in_registers(const StepParams& P, const LaneView<T>& v, const EpScratch& ep,
                                                           float* a_s, const int* pos_s) {
  const int tid = threadIdx.x, L = v.L;
  const float* lg = P.logits + ((long long)v.lane_local * P.logit_rows + row0_of<kLoop>(P, v)) * P.cap;
  float sx[E][G];
#pragma unroll
  for (int u = 0; u < E; ++u) {
    const int i = tid + u * NT;
#pragma unroll
    for (int g = 0; g < G; ++g) sx[u][g] = i < L ? __ldcg(lg + (long long)g * P.cap + i) : -INFINITY;
  }
  if (P.block_tokens > 0) {
    // Blocked prompt tail: the parked logits were taken against the cache as it was before the block.  An entry that
    // joined inside the block (its position says so) has its logit in the small table of the block's own keys.
    const int t0 = v.t - step_of<kLoop>(P, v);
    const float* lx = P.lgx + ((long long)v.lane_local * P.logit_rows + row0_of<kLoop>(P, v)) * P.block_tokens;
#pragma unroll
    for (int u = 0; u < E; ++u) {
      const int i = tid + u * NT;
      if (i < L && pos_s[i] >= t0) {
#pragma unroll
        for (int g = 0; g < G; ++g)
          sx[u][g] = kLoop ? v.lgx_s[(v.row0 + g) * P.block_tokens + (pos_s[i] - t0)] : __ldcg(lx + g * P.block_tokens + (pos_s[i] - t0));
      }
    }
    // no split partials here: the maximum of every head comes from the logits themselves (exact, order-free)
    float mx[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      mx[g] = -INFINITY;
#pragma unroll
      for (int u = 0; u < E; ++u) mx[g] = fmaxf(mx[g], sx[u][g]);
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) mx[g] = fmaxf(mx[g], __shfl_xor_sync(0xffffffffu, mx[g], off));
      if ((tid & 31) == 0) ep.w[g * kMaxSplits + (tid >> 5)] = mx[g];
    }
    group_sync<NT>();
    if (tid < G) {
      float m = ep.w[tid * kMaxSplits];
      for (int w = 1; w < NT / 32; ++w) m = fmaxf(m, ep.w[tid * kMaxSplits + w]);
      ep.M[tid] = m;
    }
    group_sync<NT>();
  } else {
    combine_partials<T, D, G, NT>(P, v, ep);
  }
  // (3) e = exp(s - M) in place, Z_g as an exact integer sum
  float Zr[G];
  {
    unsigned long long zl[G];
#pragma unroll
    for (int g = 0; g < G; ++g) zl[g] = 0ull;
#pragma unroll
    for (int u = 0; u < E; ++u) {
      if (tid + u * NT < L) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const float e = repro_exp(__fsub_rn(sx[u][g], ep.M[g]));
          sx[u][g] = e;
          zl[g] += __float2ull_rz(__fmul_rn(e, 1099511627776.0f));
        }
      }
    }
    group_sum_u64<G, NT, false>(zl, ep.u64);
#pragma unroll
    for (int g = 0; g < G; ++g) Zr[g] = __fmul_rn(__ull2float_rn(zl[g]), 1.0f / 1099511627776.0f);
  }
  // (4) probabilities, score fold, pick
  const bool compress = L > P.budget;                 // Algorithm 1's trigger: the list is longer than m
  unsigned long long best = ~0ull;
  int best_slot = -1;
  float* a_l = P.a + v.lane * P.cap;
  int32_t* pos_l = P.pos + v.lane * P.cap;
#pragma unroll
  for (int u = 0; u < E; ++u) {
    const int i = tid + u * NT;
    if (i < L) fold_one<T, G, kLoop>(P, v, a_l, pos_l, i, sx[u], Zr, a_s[i], pos_s[i], compress, best, best_slot, a_s);
  }
  clear_probs_tail<G, NT>(P, v.lane_local, row0_of<kLoop>(P, v), L);
  int j_slot;
  const unsigned long long bmin = group_min_key<NT>(best, best_slot, ep.u64 + 64, j_slot);   // its barrier also publishes a, pos
  // (5), (6)
  finish_lane<T, D, G, NT, kLoop>(P, v, ep, compress, bmin, j_slot, a_s, pos_s);
}

// ------------------------------------------------------------------------------------------------
// Kernels A1 + A2: any split count, two launches.  A1 scans: one CTA per unit, logits and partials to global
// scratch, nothing else -- its CTAs are short-lived and all alike, which keeps HBM busy.  A2 runs one CTA per lane
// on the finished scratch: o_t, probabilities, score fold, pick, merge, relink.
// ------------------------------------------------------------------------------------------------
// The scan under the even deal: CTA = (lane, unit).
template <typename T, int D, int G>
__device__ __forceinline__ void scan_body_even(const StepParams& P) {
  using C = Cfg<T, D, G>;
  constexpr int kStages = C::kStages;
  constexpr int NT = kThreads;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const Smem<T, D, G> sm(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane_id = tid & 31;
  const int split = blockIdx.x % P.n_splits;
  const int lane_local = blockIdx.x / P.n_splits;
  const int b = lane_local / P.n_kv_heads, hk = lane_local % P.n_kv_heads;
  // Ordering against the kernel launched just before this one (P.wait_at_start, chosen by the host):
  //   2  wait right here: the predecessor may touch this layer's lanes (same layer twice in a row, reset, ...).
  //   1  the predecessor works on other memory, but the caller's q, k, v may come from it: set up, read the lane's
  //      state and put the first K/V tiles in flight, then wait before the first read of a caller input.
  //   0  the caller has handed over all layers of a step at once (wkv_decode_step_layers): the predecessor is the lane
  //      epilogue of the previous layer (other lanes, other scratch set); scan alongside it and wait only at the very
  //      end, before the unit reports to its lane's epilogue, so that the completion of this grid -- and any report of
  //      it -- still implies the completion of everything before it and later kernels need not reason about more than
  //      one predecessor.
  if (P.wait_at_start == 2) griddep_wait();
  griddep_launch();
  if (P.wait_at_start == 1 && P.seq_lens != nullptr) griddep_wait();     // seq_lens is a caller input
  if (P.seq_lens != nullptr && P.tok_idx >= P.seq_lens[b]) {            // sequence already consumed (ragged prefill)
    if (P.wait_at_start != 2) griddep_wait();
    return;
  }
  LaneView<T> v;
  {
    const int* st = P.lane_state + ((long long)P.lane0 + lane_local) * LS_STRIDE;
    fill_view<T, D>(v, P, lane_local, split, st[LS_LEN], st[LS_T], st[LS_FREE]);
  }
  v.new_k = sm.aux_k(0);
  v.new_v = sm.aux_v(0);
  const T* q_in = reinterpret_cast<const T*>(P.q) + b * P.q_bs + (long long)hk * G * D;
  const T* k_in = reinterpret_cast<const T*>(P.k) + b * P.kv_bs + (long long)hk * D;
  const T* v_in = reinterpret_cast<const T*>(P.v) + b * P.kv_bs + (long long)hk * D;
  if (tid == 32 && v.slot_end > v.slot_begin) {
    // The epilogue kernel reads a and pos of these slots: pull their lines into L2 now.
    const uint32_t bytes = (uint32_t)(((v.slot_end - v.slot_begin) * 4 + 15) & ~15);   // cap is a multiple of 4 slots
    l2_prefetch(P.a + v.lane * P.cap + v.slot_begin, bytes);
    l2_prefetch(P.pos + v.lane * P.cap + v.slot_begin, bytes);
  }
  // The producer thread sets the ring up and fills every stage once; none of that reads a caller input.
  auto issue_tile = [&](int i) {
    const int s = i % kStages;
    const int slot0 = (v.tile_begin + i) * kTileSlots;
    fill_stage<T, D, G>(sm.ring + (size_t)s * C::kStageBytes, v.Kl + (long long)slot0 * D, v.Vl + (long long)slot0 * D,
                        min(kTileSlots, v.L - slot0), &sm.full_bar[s], P.vmap, (int)(v.lane * P.cap) + slot0);
  };
  if (tid == kConsumerWarps * 32) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.full_bar[s], 1);
      mbar_init(&sm.empty_bar[s], kConsumerWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    for (int i = 0; i < min(v.n_tiles, kStages); ++i) issue_tile(i);
  }
  if (P.wait_at_start == 1) griddep_wait();
  // The new token's rows are kept in shared memory for the scan (the cache copy of that slot may still be in flight)
  // and written to the cache by the CTA whose chunk owns the slot.
  for (int c = tid; c < D; c += NT) {
    sm.aux_k(0)[c] = k_in[c];
    sm.aux_v(0)[c] = v_in[c];
  }
  if (v.new_slot >= v.slot_begin && v.new_slot < v.slot_end) {
    T* Kw = const_cast<T*>(v.Kl) + (long long)v.new_slot * D;
    T* Vw = const_cast<T*>(v.Vl) + (long long)v.new_slot * D;
    for (int c = tid; c < D; c += NT) { Kw[c] = k_in[c]; Vw[c] = v_in[c]; }
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    if (lane_id == 0) {                                   // producer: keeps the ring full
      for (int i = kStages; i < v.n_tiles; ++i) {
        mbar_wait(&sm.empty_bar[i % kStages], ((i / kStages) - 1) & 1, P.status);
        issue_tile(i);
      }
    }
  } else {
    Scanner<T, D, G> sc;
    sc.begin(q_in);
    float* lg = P.logits + (long long)lane_local * G * P.cap;
    for (int i = 0; i < v.n_tiles; ++i) {
      const int s = i % kStages;
      mbar_wait(&sm.full_bar[s], (i / kStages) & 1, P.status);
      T* tK = reinterpret_cast<T*>(sm.ring + (size_t)s * C::kStageBytes);
      T* tV = reinterpret_cast<T*>(sm.ring + (size_t)s * C::kStageBytes + C::kTileBytes);
      sc.tile(tK, tV, (v.tile_begin + i) * kTileSlots, v.L, v.new_slot, v.new_k, v.new_v, P.scale, lg, P.cap, 0);
      release_stage(&sm.empty_bar[s]);
    }
    sc.end(sm.warp_part);
  }
  __syncthreads();
  combine_warps<D, G, NT>(sm.warp_part, P.part + ((long long)lane_local * P.n_splits + split) * G * (D + 2));
  // Level 0: the wait comes BEFORE the unit reports.  The lane epilogues behind this scan start on the reports alone,
  // and the scan after them (which reuses the scratch set of the lane epilogues in front of this scan) is released by
  // those epilogues: with the report behind the wait, "the next scan runs" implies "every unit here has seen the
  // previous lane epilogues complete", so no two grids ever touch one scratch set at a time.
  if (!P.wait_at_start) griddep_wait();
  if (P.ticket != nullptr) {
    // tell the lane's epilogue CTA (already resident in the next kernel, or not yet) that this unit is in scratch
    __syncthreads();
    if (tid == 0) {
      __threadfence();                                   // release: the barrier ordered every thread's stores before it
      atomicAdd(&P.ticket[lane_local], 1u);
    }
  }
}

// The scan under either deal as a loop over the CTA's pieces; compiled for the flat deal (kFlat, P.flat_chunk > 0): the
// even deal's single pass above carries no loop state and starts a little faster, which 2560 short CTAs per launch feel.
template <typename T, int D, int G, bool kFlat>
__device__ __forceinline__ void scan_body(const StepParams& P) {
  using C = Cfg<T, D, G>;
  constexpr int kStages = C::kStages;
  constexpr int NC = kConsumerWarps * 32;               // consumer threads: 0 .. NC-1; thread NC is the producer
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const Smem<T, D, G> sm(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane_id = tid & 31;
  // Ordering against the kernel launched just before this one (P.wait_at_start, chosen by the host):
  //   2  wait right here: the predecessor may touch this layer's lanes (same layer twice in a row, reset, ...).
  //   1  the predecessor works on other memory, but the caller's q, k, v may come from it: set up, read the lanes'
  //      state and put the first K/V tiles in flight, then wait before the first read of a caller input.
  //   0  the caller has handed over all layers of a step at once (wkv_decode_step_layers): the predecessor is the lane
  //      epilogue of the previous layer (other lanes, other scratch set); scan alongside it and wait only at the very
  //      end, before the unit reports to its lane's epilogue, so that the completion of this grid -- and any report of
  //      it -- still implies the completion of everything before it and later kernels need not reason about more than
  //      one predecessor.
  if (P.wait_at_start == 2) griddep_wait();
  griddep_launch();
  if (P.wait_at_start == 1 && P.seq_lens != nullptr) griddep_wait();     // seq_lens is a caller input
  // the lanes this CTA works on: one under the even deal, one or more (a piece of each) under the flat deal
  int lane_lo, lane_hi;
  if constexpr (!kFlat) {
    lane_lo = lane_hi = blockIdx.x / P.n_splits;
  } else {
    const long long g0 = (long long)blockIdx.x * P.flat_chunk;
    const long long g1 = min(g0 + P.flat_chunk, (long long)P.n_lanes * P.tiles_cap);
    lane_lo = (int)(g0 / P.tiles_cap);
    lane_hi = g1 > g0 ? (int)((g1 - 1) / P.tiles_cap) : lane_lo - 1;
  }
  // the view of one of those lanes and this CTA's share of it; false: the lane's sequence is already consumed (ragged prefill)
  auto view_of = [&](int lane_local, LaneView<T>& v) -> bool {
    const int b = lane_local / P.n_kv_heads;
    if (P.seq_lens != nullptr && P.tok_idx >= P.seq_lens[b]) return false;
    const int* st = P.lane_state + ((long long)P.lane0 + lane_local) * LS_STRIDE;
    fill_view<T, D>(v, P, lane_local, kFlat ? 0 : (int)(blockIdx.x % P.n_splits), st[LS_LEN], st[LS_T], st[LS_FREE]);
    if constexpr (kFlat) flat_piece(v, P, lane_local, (int)blockIdx.x);
    v.new_k = sm.aux_k(0);
    v.new_v = sm.aux_v(0);
    return true;
  };
  // The producer warp sets the ring's barriers up, says so on a named barrier without waiting there, and starts filling
  // the ring at once; the consumer warps wait on that named barrier before their first look at the ring.
  if (warp == kConsumerWarps) {
    if (lane_id == 0) {
      for (int s = 0; s < kStages; ++s) {
        mbar_init(&sm.full_bar[s], 1);
        mbar_init(&sm.empty_bar[s], kConsumerWarps);
      }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    asm volatile("bar.arrive 2, %0;" ::"n"(kThreads) : "memory");
    if (lane_id == 0) {
      // Producer: keeps the ring full across the CTA's pieces.  It reads lane state and cache rows only, none of which
      // the kernel in front of this one writes, so it does not wait for that kernel (levels 0 and 1).
      int it = 0;                                           // tiles issued so far, over all pieces
      int lane_local = lane_lo;
      if (lane_lo <= lane_hi) do {
        LaneView<T> v;
        if (!view_of(lane_local, v)) continue;
        if (v.slot_end > v.slot_begin) {
          // The epilogue kernel reads a and pos of these slots: pull their lines into L2 now.
          const uint32_t bytes = (uint32_t)(((v.slot_end - v.slot_begin) * 4 + 15) & ~15);   // cap is a multiple of 4 slots
          l2_prefetch(P.a + v.lane * P.cap + v.slot_begin, bytes);
          l2_prefetch(P.pos + v.lane * P.cap + v.slot_begin, bytes);
        }
        for (int i = 0; i < v.n_tiles; ++i, ++it) {
          const int s = it % kStages;
          if (it >= kStages) mbar_wait(&sm.empty_bar[s], ((it / kStages) - 1) & 1, P.status);
          const int slot0 = (v.tile_begin + i) * kTileSlots;
          fill_stage<T, D, G>(sm.ring + (size_t)s * C::kStageBytes, v.Kl + (long long)slot0 * D, v.Vl + (long long)slot0 * D,
                              min(kTileSlots, v.L - slot0), &sm.full_bar[s], P.vmap, (int)(v.lane * P.cap) + slot0);
        }
      } while (kFlat && ++lane_local <= lane_hi);
    }
  } else {
    if (P.wait_at_start == 1) griddep_wait();             // before the first read of q, k, v
    asm volatile("bar.sync 2, %0;" ::"n"(kThreads) : "memory");   // the ring's barriers exist
    int it = 0;                                           // tiles consumed so far, over all pieces
    int lane_local = lane_lo;
    if (lane_lo <= lane_hi) do {
      LaneView<T> v;
      if (!view_of(lane_local, v)) continue;
      const int b = v.b, hk = v.hk;
      const T* q_in = reinterpret_cast<const T*>(P.q) + b * P.q_bs + (long long)hk * G * D;
      const T* k_in = reinterpret_cast<const T*>(P.k) + b * P.kv_bs + (long long)hk * D;
      const T* v_in = reinterpret_cast<const T*>(P.v) + b * P.kv_bs + (long long)hk * D;
      // The new token's rows are kept in shared memory for the scan (the cache copy of that slot may still be in
      // flight) and written to the cache by the CTA whose share owns the slot.  (The barrier at the end of the previous
      // piece has every consumer warp done with the previous lane's rows.)
      for (int c = tid; c < D; c += NC) {
        sm.aux_k(0)[c] = k_in[c];
        sm.aux_v(0)[c] = v_in[c];
      }
      if (v.new_slot >= v.slot_begin && v.new_slot < v.slot_end) {
        T* Kw = const_cast<T*>(v.Kl) + (long long)v.new_slot * D;
        T* Vw = const_cast<T*>(v.Vl) + (long long)v.new_slot * D;
        for (int c = tid; c < D; c += NC) { Kw[c] = k_in[c]; Vw[c] = v_in[c]; }
      }
      group_sync<NC>();
      Scanner<T, D, G> sc;
      sc.begin(q_in);
      float* lg = P.logits + (long long)lane_local * G * P.cap;
      for (int i = 0; i < v.n_tiles; ++i, ++it) {
        const int s = it % kStages;
        mbar_wait(&sm.full_bar[s], (it / kStages) & 1, P.status);
        T* tK = reinterpret_cast<T*>(sm.ring + (size_t)s * C::kStageBytes);
        T* tV = reinterpret_cast<T*>(sm.ring + (size_t)s * C::kStageBytes + C::kTileBytes);
        sc.tile(tK, tV, (v.tile_begin + i) * kTileSlots, v.L, v.new_slot, v.new_k, v.new_v, P.scale, lg, P.cap, 0);
        release_stage(&sm.empty_bar[s]);
      }
      sc.end(sm.warp_part);
      group_sync<NC>();
      combine_warps<D, G, NC>(sm.warp_part, P.part + ((long long)lane_local * P.n_splits + v.split) * G * (D + 2));
      // Level 0: the wait comes BEFORE the unit reports.  The lane epilogues behind this scan start on the reports
      // alone, and the scan after them (which reuses the scratch set of the lane epilogues in front of this scan) is
      // released by those epilogues: with the report behind the wait, "the next scan runs" implies "every unit here has
      // seen the previous lane epilogues complete", so no two grids ever touch one scratch set at a time.
      if (!P.wait_at_start) griddep_wait();
      // the barrier orders every consumer's stores (partial, logits, cache row) before the report, and ends the piece:
      // the next piece may overwrite the token rows and the warp partials
      group_sync<NC>();
      if (P.ticket != nullptr && tid == 0) {
        // tell the lane's epilogue CTA (already resident in the next kernel, or not yet) that this unit is in scratch
        __threadfence();                                 // release
        atomicAdd(&P.ticket[lane_local], 1u);
      }
    } while (kFlat && ++lane_local <= lane_hi);
  }
  // every CTA, with work or without, ends behind the kernel in front of it: the completion of this grid implies that
  // kernel's completion
  if (P.wait_at_start != 2) griddep_wait();
}

template <typename T, int D, int G, bool kFlat>
__global__ void __launch_bounds__(kThreads) scan_kernel(const __grid_constant__ StepParams P) {
  if constexpr (kFlat) scan_body<T, D, G, true>(P);
  else scan_body_even<T, D, G>(P);
}
// The same scan for the instantiations with the tensor-core P.V half (Cfg::kMmaPV), held to the registers of four CTAs
// per SM (a second argument to __launch_bounds__ changes the compiler's choices even when it is 1, hence two entries).
template <typename T, int D, int G, bool kFlat>
__global__ void __launch_bounds__(kThreads, 4) scan_kernel_mma(const __grid_constant__ StepParams P) {
  if constexpr (kFlat) scan_body<T, D, G, true>(P);
  else scan_body_even<T, D, G>(P);
}
// the entry that a configuration's scan is launched through
template <typename T, int D, int G>
inline auto scan_entry(bool flat) -> void (*)(const StepParams) {
  if constexpr (Cfg<T, D, G>::kMmaPV) return flat ? scan_kernel_mma<T, D, G, true> : scan_kernel_mma<T, D, G, false>;
  else return flat ? scan_kernel<T, D, G, true> : scan_kernel<T, D, G, false>;
}
// dynamic shared memory of that entry
template <typename T, int D, int G>
constexpr int scan_smem_bytes() { return Cfg<T, D, G>::kScanBytes; }

constexpr int kEpilogueThreads = 256;
constexpr int kEpilogueThreadsMid = 384;      // four query heads, a layer of at most two lanes per SM
constexpr int kEpilogueThreadsWide = 512;     // one or two query heads only (registers: two CTAs per SM)
// Slots per thread that the register version of the lane epilogue is compiled for (0: not compiled); a thread keeps
// E * G logits in registers.  17 x 256 and 9 x 512 threads cover the 4097 entries of the largest single-head workload,
// 9 x 384 the 3278 entries of the grouped-query one.
__host__ __device__ constexpr int epilogue_slots_per_thread(int G, int NT) {
  return G == 1 ? (NT >= 512 ? 9 : 17) : G == 2 ? (NT >= 512 ? 5 : 9) : (G == 4 && NT >= 384) ? 9 : 0;
}

// NT threads per lane: kEpilogueThreads, or kEpilogueThreadsWide when a layer has so few lanes that two wide CTAs per
// SM still hold them all -- the epilogue is a chain of load -> compute rounds, and twice the threads halve the rounds.
template <typename T, int D, int G, int NT>
__device__ __forceinline__ void lane_epilogue_body(const StepParams& P) {
  __shared__ __align__(16) unsigned char ep_raw[EpScratch::bytes(G)];
  EpScratch ep;
  ep.carve(ep_raw, G);
  const int lane_local = blockIdx.x;
  const int b = lane_local / P.n_kv_heads, hk = lane_local % P.n_kv_heads;
  const bool active = !(P.seq_lens != nullptr && P.tok_idx >= P.seq_lens[b]);   // else: sequence already consumed
  // The lane's state words were last written by an earlier lane epilogue of the same layer, which is complete (the
  // scan in front of this kernel did not finish before everything older had finished): read them before waiting.
  // (A step of a blocked prompt tail follows the previous step of the same lanes: nothing is read before that one is done.)
  if (P.block_tokens > 0) griddep_wait();
  LaneView<T> v;
  const int* st = P.lane_state + ((long long)P.lane0 + lane_local) * LS_STRIDE;
  if (active) {
    fill_view<T, D>(v, P, lane_local, 0, st[LS_LEN], st[LS_T], st[LS_FREE]);
    v.head = st[LS_HEAD];
    v.tail = st[LS_TAIL];
    v.new_k = v.Kl + (long long)v.new_slot * D;          // the scan kernel has stored this step's token in the cache
    v.new_v = v.Vl + (long long)v.new_slot * D;
    if (P.block_tokens > 0) {
      // ... in a blocked tail no scan runs per token: the token's rows go into its slot here.  (Thread c writes channel c
      // and is the only one to read it back from the cache in this kernel.)
      const T* k_in = reinterpret_cast<const T*>(P.k) + b * P.kv_bs + (long long)hk * D;
      const T* v_in = reinterpret_cast<const T*>(P.v) + b * P.kv_bs + (long long)hk * D;
      for (int c = threadIdx.x; c < D; c += NT) {
        const_cast<T*>(v.new_k)[c] = k_in[c];
        const_cast<T*>(v.new_v)[c] = v_in[c];
      }
    }
  }
  // A lane of at most E * NT entries is finished by lane_epilogue_in_registers, if the launch gave the CTA room to stage
  // the lane's scores and positions (P.ep_stage_slots entries each of dynamic shared memory).  They were last written
  // where its state words were, so they too can be fetched before waiting; the entry of this step's token starts from
  // a = 0 (Algorithm 1's [a, 0]) at position t.
  constexpr int E = epilogue_slots_per_thread(G, NT);
  extern __shared__ __align__(16) unsigned char ep_dyn[];
  float* a_s = reinterpret_cast<float*>(ep_dyn);
  int* pos_s = reinterpret_cast<int*>(ep_dyn) + P.ep_stage_slots;
  const bool in_regs = E > 0 && active && v.L <= E * NT && v.L <= P.ep_stage_slots;
  if (in_regs) {
    const float* a_l = P.a + v.lane * P.cap;
    const int32_t* pos_l = P.pos + v.lane * P.cap;
    for (int i = threadIdx.x; i < v.L; i += NT) {
      const bool old_entry = i != v.new_slot;
      a_s[i] = old_entry ? __ldcg(a_l + i) : 0.f;
      pos_s[i] = old_entry ? __ldcg(pos_l + i) : v.t;
    }
  }
  // When is the lane's scan in scratch?  Without tickets: when the whole scan kernel has completed.  With tickets: as
  // soon as the lane's own n_splits units have reported -- this kernel's CTAs become resident only after every CTA of
  // the scan has started (that is the launch condition), so the units being waited for are running or done and never
  // depend on this kernel; the wait is bounded all the same.
  if (P.ticket == nullptr || !active) {
    griddep_wait();
    griddep_launch();
    if (!active) {
      if (threadIdx.x == 0 && P.evicted) P.evicted[b * P.ev_bs + hk] = -1;
      return;
    }
  } else {
    if (threadIdx.x == 0) {
      volatile uint32_t* tk = P.ticket + lane_local;
      int first_cta, n_pieces;
      lane_pieces(P, lane_local, first_cta, n_pieces);
      int ok = 0;
      for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (*tk >= (uint32_t)n_pieces) { ok = 1; break; }
        __nanosleep(100);
      }
      if (!ok) atomicOr(P.status, kStatusWaitTimeout);
      __threadfence();                                   // acquire side of the units' release
      ep.i32[5] = ok;
    }
    __syncthreads();
    griddep_launch();                                    // the next kernel in the stream may be set up alongside
    if (!ep.i32[5]) {                                    // gave up: leave the lane untouched, the status word says so
      griddep_wait();
      return;
    }
  }
  if (in_regs) {
    if constexpr (E > 0) lane_epilogue_in_registers<T, D, G, NT, E>(P, v, ep, a_s, pos_s);
  } else if (P.block_tokens > 0) {
    if (threadIdx.x == 0) atomicOr(P.status, kStatusBadLink);   // the host sends blocked tails only where the lane fits
  } else {
    lane_epilogue_from_scratch<T, D, G, NT>(P, v, ep);
  }
  if (P.ticket != nullptr) {
    if (threadIdx.x == 0) P.ticket[lane_local] = 0u;     // ready for the next call that uses this scratch set
    griddep_wait();                                      // keeps "this grid complete => the scan complete" literally true
  }
}

// One query head: held to 64 registers, i.e. 1024 threads per SM, so that a layer of up to 4 x 148 lanes is one wave of
// CTAs -- the kernel behind this one can only be set up once every CTA here has started, and a second wave would start
// only when the first has finished.
template <typename T, int D, int G, int NT>
__global__ void __launch_bounds__(NT, G == 1 ? 1024 / NT : 1) lane_epilogue_kernel(const StepParams P) {
  lane_epilogue_body<T, D, G, NT>(P);
}
// The per-token lane epilogue for a whole block of a blocked prompt tail in ONE launch: a lane's tokens follow one another
// inside the lane's CTA (lanes are independent, so nothing is ordered across CTAs), which spares the launch gap and the
// grid-wide wait between tokens that one launch per token costs.  Same steps, same order, same results as B launches of
// lane_epilogue_kernel with block_step = 0 .. B-1.
template <typename T, int D, int G, int NT>
__device__ __forceinline__ void lane_epilogue_block_body(const StepParams& P) {
  __shared__ __align__(16) unsigned char ep_raw[EpScratch::bytes(G)];
  EpScratch ep;
  ep.carve(ep_raw, G);
  constexpr int E = epilogue_slots_per_thread(G, NT);
  extern __shared__ __align__(16) unsigned char ep_dyn[];
  float* a_s = reinterpret_cast<float*>(ep_dyn);
  int* pos_s = reinterpret_cast<int*>(ep_dyn) + P.ep_stage_slots;
  const int lane_local = blockIdx.x;
  const int b = lane_local / P.n_kv_heads, hk = lane_local % P.n_kv_heads;
  griddep_wait();                                        // the block's logit sweep (and everything before it) is done
  griddep_launch();
  // What a token's step would otherwise fetch from L2 again is kept in shared memory from token to token: the lane's
  // state words (thread 0 keeps the copy current), its scores and positions (staged once; every step's fold keeps
  // the scores current, and the only position that changes is the new token's) and the block's own-key logits.
  __shared__ int st_s[LS_STRIDE];
  __shared__ float lgx_s[64];                            // rows * block_tokens = G * B * B <= 64
  {
    const int* st = P.lane_state + ((long long)P.lane0 + lane_local) * LS_STRIDE;
    if (threadIdx.x < LS_STRIDE) st_s[threadIdx.x] = __ldcg(st + threadIdx.x);
    const int n_lgx = min(64, P.logit_rows * P.block_tokens);
    for (int i = threadIdx.x; i < n_lgx; i += NT) lgx_s[i] = __ldcg(P.lgx + (long long)lane_local * P.logit_rows * P.block_tokens + i);
  }
  __syncthreads();
  bool staged = false;
  for (int step = 0; step < P.block_n; ++step) {
    if (P.seq_lens != nullptr && P.tok_idx + step >= P.seq_lens[b]) {          // the sequence has ended (same for the whole CTA)
      if (threadIdx.x == 0 && P.evicted) P.evicted[b * P.ev_bs + hk + (long long)step * P.ev_ts] = -1;
      continue;
    }
    LaneView<T> v;
    fill_view<T, D>(v, P, lane_local, 0, st_s[LS_LEN], st_s[LS_T], st_s[LS_FREE]);   // written by thread 0 in the step before
    v.head = st_s[LS_HEAD];
    v.tail = st_s[LS_TAIL];
    v.step = step;
    v.row0 = step * G;
    v.st_s = st_s;
    v.lgx_s = lgx_s;
    v.new_k = v.Kl + (long long)v.new_slot * D;
    v.new_v = v.Vl + (long long)v.new_slot * D;
    {
      // the token's rows go into its slot (thread c writes channel c and is the only one to read it back in this step)
      const T* k_in = reinterpret_cast<const T*>(P.k) + b * P.kv_bs + (long long)step * P.kv_ts + (long long)hk * D;
      const T* v_in = reinterpret_cast<const T*>(P.v) + b * P.kv_bs + (long long)step * P.kv_ts + (long long)hk * D;
      for (int c = threadIdx.x; c < D; c += NT) {
        const_cast<T*>(v.new_k)[c] = k_in[c];
        const_cast<T*>(v.new_v)[c] = v_in[c];
      }
    }
    if (E > 0 && v.L <= E * NT && v.L <= P.ep_stage_slots) {
      if (!staged) {
        const float* a_l = P.a + v.lane * P.cap;
        const int32_t* pos_l = P.pos + v.lane * P.cap;
        for (int i = threadIdx.x; i < v.L; i += NT) {
          const bool old_entry = i != v.new_slot;
          a_s[i] = old_entry ? __ldcg(a_l + i) : 0.f;
          pos_s[i] = old_entry ? __ldcg(pos_l + i) : v.t;
        }
        staged = true;
      } else if ((int)threadIdx.x == v.new_slot % NT) {    // the thread that owns the slot: Algorithm 1's [a, 0] at position t
        a_s[v.new_slot] = 0.f;
        pos_s[v.new_slot] = v.t;
      }
      if constexpr (E > 0) lane_epilogue_in_registers<T, D, G, NT, E, true>(P, v, ep, a_s, pos_s);
    } else if (threadIdx.x == 0) {
      atomicOr(P.status, kStatusBadLink);                 // the host sends blocked tails only where the lane fits
    }
    __syncthreads();                                     // the step's writes before the next step reads them; scratch reuse
  }
}
template <typename T, int D, int G, int NT>
__global__ void __launch_bounds__(NT, G == 1 ? 1024 / NT : 1) lane_epilogue_block_kernel(const StepParams P) {
  lane_epilogue_block_body<T, D, G, NT>(P);
}
template <typename T, int D, int G>
__global__ void __launch_bounds__(kEpilogueThreadsMid, 2) lane_epilogue_block_kernel_mid(const StepParams P) {
  lane_epilogue_block_body<T, D, G, kEpilogueThreadsMid>(P);
}

// Four query heads, a layer of at most two lanes per SM: 384 threads per lane, held to the registers of two CTAs per SM.
template <typename T, int D, int G>
__global__ void __launch_bounds__(kEpilogueThreadsMid, 2) lane_epilogue_kernel_mid(const StepParams P) {
  lane_epilogue_body<T, D, G, kEpilogueThreadsMid>(P);
}

// ------------------------------------------------------------------------------------------------
// Kernel B: the n_splits CTAs of a lane form one thread-block cluster.  Cluster barriers are hardware barriers among
// co-scheduled CTAs; every CTA of an active lane reaches every barrier.
// ------------------------------------------------------------------------------------------------
template <typename T, int D, int G>
__global__ void __launch_bounds__(kThreads) decode_step_cluster_kernel(const __grid_constant__ StepParams P) {
  namespace cg = cooperative_groups;
  using C = Cfg<T, D, G>;
  constexpr int kStages = C::kStages;
  constexpr int NT = kThreads;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const Smem<T, D, G> sm(smem_raw);
  const float kLog2e = 1.4426950408889634f;
  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, warp = tid >> 5, lane_id = tid & 31;
  const int S = P.n_splits;
  const int split = (int)cluster.block_rank();
  const int lane_local = blockIdx.x / S;
  const int b = lane_local / P.n_kv_heads, hk = lane_local % P.n_kv_heads;
  // Launched with programmatic stream serialization: the next kernel in the stream may be made resident as soon as
  // every CTA of this grid has started (that hides its launch latency behind this grid's tail, which matters when a
  // step is a few microseconds long); this grid touches nothing before its predecessor has completed.
  griddep_launch();
  griddep_wait();
  if (P.seq_lens != nullptr && P.tok_idx >= P.seq_lens[b]) {      // sequence already consumed: same decision in every CTA
    if (split == 0 && tid == 0 && P.evicted) P.evicted[b * P.ev_bs + hk] = -1;
    return;
  }
  LaneView<T> v;
  {
    const int* st = P.lane_state + ((long long)P.lane0 + lane_local) * LS_STRIDE;
    fill_view<T, D>(v, P, lane_local, split, st[LS_LEN], st[LS_T], st[LS_FREE]);
  }
  v.new_k = sm.aux_k(0);
  v.new_v = sm.aux_v(0);
  const T* q_in = reinterpret_cast<const T*>(P.q) + b * P.q_bs + (long long)hk * G * D;
  const T* k_in = reinterpret_cast<const T*>(P.k) + b * P.kv_bs + (long long)hk * D;
  const T* v_in = reinterpret_cast<const T*>(P.v) + b * P.kv_bs + (long long)hk * D;
  const int n_mine = v.slot_end - v.slot_begin;
  if (split == 0) { v.head = v.st[LS_HEAD]; v.tail = v.st[LS_TAIL]; }

  if (tid == 32 && n_mine > 0) {
    // The epilogue reads a and pos of these slots long after the scan: pull their lines into L2 now.
    const uint32_t bytes = (uint32_t)((n_mine * 4 + 15) & ~15);          // cap is a multiple of 4 slots
    l2_prefetch(P.a + v.lane * P.cap + v.slot_begin, bytes);
    l2_prefetch(P.pos + v.lane * P.cap + v.slot_begin, bytes);
  }
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.full_bar[s], 1);
      mbar_init(&sm.empty_bar[s], kConsumerWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // The new token's rows are kept in shared memory for the scan (the cache copy of that slot may still be in flight)
  // and written to the cache by the CTA whose chunk owns the slot.
  for (int c = tid; c < D; c += NT) {
    sm.aux_k(0)[c] = k_in[c];
    sm.aux_v(0)[c] = v_in[c];
  }
  if (v.new_slot >= v.slot_begin && v.new_slot < v.slot_end) {
    T* Kw = const_cast<T*>(v.Kl) + (long long)v.new_slot * D;
    T* Vw = const_cast<T*>(v.Vl) + (long long)v.new_slot * D;
    for (int c = tid; c < D; c += NT) { Kw[c] = k_in[c]; Vw[c] = v_in[c]; }
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    if (lane_id == 0) {                                   // producer: keeps the ring full
      for (int i = 0; i < v.n_tiles; ++i) {
        const int s = i % kStages;
        if (i >= kStages) mbar_wait(&sm.empty_bar[s], ((i / kStages) - 1) & 1, P.status);
        const int slot0 = (v.tile_begin + i) * kTileSlots;
        fill_stage<T, D, G>(sm.ring + (size_t)s * C::kStageBytes, v.Kl + (long long)slot0 * D,
                            v.Vl + (long long)slot0 * D, min(kTileSlots, v.L - slot0), &sm.full_bar[s], P.vmap,
                            (int)(v.lane * P.cap) + slot0);
      }
    }
  } else {
    Scanner<T, D, G> sc;
    sc.begin(q_in);
    for (int i = 0; i < v.n_tiles; ++i) {
      const int s = i % kStages;
      mbar_wait(&sm.full_bar[s], (i / kStages) & 1, P.status);
      T* tK = reinterpret_cast<T*>(sm.ring + (size_t)s * C::kStageBytes);
      T* tV = reinterpret_cast<T*>(sm.ring + (size_t)s * C::kStageBytes + C::kTileBytes);
      sc.tile(tK, tV, (v.tile_begin + i) * kTileSlots, v.L, v.new_slot, v.new_k, v.new_v, P.scale, sm.chunk_logits,
              P.chunk_cap, v.slot_begin);
      release_stage(&sm.empty_bar[s]);
    }
    sc.end(sm.warp_part);
  }
  __syncthreads();
  combine_warps<D, G, NT>(sm.warp_part, sm.cta_part);
  cluster.sync();                                       // #1: every CTA's partial is readable

  // (1) global max per head (every CTA), output weights (rank 0)
  if (tid < G) {
    const int g = tid;
    float M = -INFINITY;
    for (int s = 0; s < S; ++s) M = fmaxf(M, cluster.map_shared_rank(sm.cta_part, s)[g * (D + 2)]);
    sm.ep.M[g] = M;
    if (split == 0) {
      float lsum = 0.f;
      for (int s = 0; s < S; ++s) {
        const float* pp = cluster.map_shared_rank(sm.cta_part, s) + g * (D + 2);
        const float w = fast_exp2((pp[0] - M) * kLog2e);
        sm.ep.w[g * kMaxSplits + s] = w;
        lsum += w * pp[1];
      }
      sm.ep.linv[g] = 1.f / lsum;
    }
  }
  __syncthreads();
  // (2) o_t by rank 0
  if (split == 0) {
    T* out = reinterpret_cast<T*>(P.out) + v.b * P.out_bs + (long long)v.hk * G * D;
    for (int idx = tid; idx < G * D; idx += NT) {
      const int g = idx / D, c = idx % D;
      float o = 0.f;
      for (int s = 0; s < S; ++s) o += sm.ep.w[g * kMaxSplits + s] * cluster.map_shared_rank(sm.cta_part, s)[g * (D + 2) + 2 + c];
      out[idx] = from_f32<T>(o * sm.ep.linv[g]);
    }
  }
  // (3) this CTA's share of Z
  {
    unsigned long long zl[G];
    exp_and_zsum<G, false, NT>(sm.chunk_logits, P.chunk_cap, n_mine, sm.ep.M, zl);
    group_sum_u64<G, NT>(zl, sm.ep.u64);
    if (tid == 0) {
#pragma unroll
      for (int g = 0; g < G; ++g) sm.ep.u64[96 + g] = zl[g];
    }
  }
  cluster.sync();                                       // #2: Z partials readable (and rank 0 is done with the o partials)
  if (tid < G) {
    unsigned long long z = 0ull;
    for (int s = 0; s < S; ++s) z += cluster.map_shared_rank(sm.ep.u64, s)[96 + tid];
    sm.ep.Z[tid] = __fmul_rn(__ull2float_rn(z), 1.0f / 1099511627776.0f);
  }
  __syncthreads();
  // (4) probabilities, score fold and pick over this CTA's slots
  const bool compress = v.L > P.budget;
  unsigned long long best = ~0ull;
  int best_slot = -1;
  fold_scores<T, G, NT>(P, v, sm.chunk_logits, P.chunk_cap, v.slot_begin, n_mine, sm.ep.Z, compress, best, best_slot);
  if (P.probs && split == S - 1) {
    for (int i = v.L + tid; i < P.budget + 1; i += NT)
#pragma unroll
      for (int g = 0; g < G; ++g)
        P.probs[((long long)v.b * P.n_kv_heads * G + (long long)v.hk * G + g) * (P.budget + 1) + i] = 0.f;
  }
  int my_slot;
  const unsigned long long my_min = group_min_key<NT>(best, best_slot, sm.ep.u64 + 64, my_slot);
  if (tid == 0) { sm.ep.u64[104] = my_min; sm.ep.i32[1] = my_slot; }
  cluster.sync();                                       // #3: keys readable; a and pos of every slot are written
  // (5) rank 0 gathers the lane's pick
  if (split == 0 && tid == 0) {
    unsigned long long bmin = ~0ull;
    int j = -1;
    for (int s = 0; s < S; ++s) {
      const unsigned long long k = cluster.map_shared_rank(sm.ep.u64, s)[104];
      if (k < bmin) { bmin = k; j = cluster.map_shared_rank(sm.ep.i32, s)[1]; }
    }
    sm.ep.i32[4] = j;
    sm.ep.u64[105] = bmin;
  }
  cluster.sync();                                       // #4: nobody's shared memory is needed any more
  if (split != 0) return;
  finish_lane<T, D, G, NT>(P, v, sm.ep, compress, sm.ep.u64[105], sm.ep.i32[4]);
}

// Exercises the give-up path of the bounded wait without any fault: one thread waits on an mbarrier that nothing
// will ever complete, runs out of polls, records that in the status word, and the kernel ends normally.
__global__ void wait_selftest_kernel(uint32_t* status, uint32_t polls) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_wait(&bar, 0, status, polls);
  }
}

// Clears a context: every lane empty, chain heads/tails unset, slot 0 free.
__global__ void reset_kernel(int32_t* lane_state, int32_t* pos, float* a, int32_t* next, int32_t* prev, long long lanes,
                             int cap, uint32_t* status) {
  const long long n = lanes * cap;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    pos[i] = -1;
    a[i] = 0.f;
    next[i] = -1;
    prev[i] = -1;
  }
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < lanes; i += (long long)gridDim.x * blockDim.x) {
    int32_t* st = lane_state + i * LS_STRIDE;
    st[LS_LEN] = 0; st[LS_T] = 0; st[LS_HEAD] = -1; st[LS_TAIL] = -1; st[LS_FREE] = 0;
    st[5] = 0; st[6] = 0; st[7] = 0;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) *status = 0u;
}

}  // namespace wkv
