// Bulk prompt phase of WeightedKV (Algorithm 1) for sm_100a.
//
// Algorithm 1 streams: one token, one pass over the cache.  While a lane holds at most `budget` entries nothing is
// compressed, so the first n = min(prompt length, budget) iterations are plain causal attention and can be done as one
// dense problem per lane: logits S = scale * Q K^T (lower triangle), row softmax, outputs O = P V, and the column sums
// a_i = sum_t mean_g P[t, g, i] that Algorithm 1 accumulates one step at a time.  This kernel computes exactly what
// those n streamed steps compute: every logit with the reproducible dot, every probability with the reproducible
// exponential and the integer-sum normaliser, and every a_i by adding its terms in ascending t, so that K, pos, a and
// the links come out bit-identical to streaming; the outputs (not part of that chain) agree to rounding.  A lane may
// already hold uncompressed tokens from earlier calls (a prompt fed in chunks): their keys and values are read from
// the cache, where token i still sits in slot i, and the new rows attend to them as well.
//
// One CTA per lane walks the prompt in blocks of 16 query rows (16 / G tokens x G query heads):
//   phase 1  S block = Q block . K^T tile by tile (fp32 FMAs in the reproducible order), causal mask, parked in an
//            L2-resident scratch row block; exact row maxima
//   phase 2  e = exp(s - M) in place, Z as an exact integer sum
//   phase 3  per key tile: P = e / Z, a_i += group mean (rows in ascending t), O += P . V (bf16 storage: tensor
//            cores, each probability as a bf16 hi + lo pair; fp32 storage: packed fp32 FMAs)
// K and V tiles arrive through a two-stage ring of bulk asynchronous copies (one row per thread, byte-counted on an
// mbarrier), issued two tiles ahead -- the V tiles of a block while its exponentials are computed, the K tiles of the
// next block while this block's outputs are stored -- so the tile loads overlap the arithmetic.
// The work is arithmetic-bound (about n^2 d G FMAs per lane against n d bytes): the roofline is the fp32 pipe.
#pragma once
#include "wkv_kernels.cuh"

namespace wkv {

constexpr int kBulkRows = 16;        // query rows per block: 16 / G tokens x G heads (kBulkRowsWide: 32, for layers of few lanes)
constexpr int kBulkRowsWide = 32;
constexpr int kBulkKeys = 128;       // granularity of the scratch rows (a multiple of every tile size)
// A CTA has 8 threads per query row of its block: warp w owns query rows 4w .. 4w+3.  A layer with at most two lanes per
// SM runs blocks of 32 rows on 256 threads: twice the warps per SM for the same registers per thread, and every key
// and value tile is fetched half as often.
__host__ __device__ constexpr int bulk_threads(int rows) { return 8 * rows; }
__host__ __device__ constexpr int bulk_pad_p(int rows) { return rows + 4; }   // floats per key in the probability tile (the rows + padding)

struct PrefillParams {
  void* Kc;
  void* Vc;
  float* a;
  int32_t* pos;
  int32_t* next;
  int32_t* prev;
  int32_t* lane_state;
  float* S;                  // [lanes of the layer][kBulkRows][s_stride] logits, then exponentials
  const void* Q;             // [batch, T_max, n_q_heads, D] ([n_layers * batch, ...] for a launch over all layers)
  const void* K;             // [batch, T_max, n_kv_heads, D]
  const void* V;
  void* out;                 // [batch, T_max, n_q_heads, D] or null
  int32_t* evicted;          // [batch, T_max, n_kv_heads] or null
  const int32_t* seq_lens;   // [batch] or null
  int batch;                 // sequences per layer: a launch over several layers indexes seq_lens by b % batch
  int lane0, n_kv_heads, cap, T_max;
  int n0;                    // tokens this kernel covers at most: min(T_max, budget)
  int s_stride;              // multiple of kBulkKeys, >= n0
  float scale;
  uint32_t* status;          // device status word (bounded waits report here)
  // 2-byte rows only: tensor maps over the K and the V cache as [lanes_total * cap][D] matrices, boxes of 64 elements x
  // one tile of keys, 128-byte swizzle (encoded once per context).
  alignas(64) unsigned char kmap[128];
  alignas(64) unsigned char vmap[128];
};

// Keys per tile (a template parameter of the kernel): 64, or 128 for 2-byte storage.  Two tiles of padded rows live in
// shared memory.  128-key tiles amortise the per-tile work better (4 x 4 outputs per thread, two CTAs per SM); 64-key
// tiles let four CTAs share an SM, which wins once a layer has more lanes than two per SM.

// 2-byte rows (kTma): a tile arrives as one tensor-map copy per 128-byte half of its rows, in the 128-byte swizzle
// ([half][key][128 B], 16-byte chunk index XORed with key % 8), instead of one bulk copy per row into padded rows: the
// copy engine of an SM takes tens of cycles per request whatever its size, and a row per request kept it busier than
// the arithmetic.  Both layouts are free of bank conflicts for the two access patterns (a thread per key in the logits,
// transposed fragment loads in P.V).  The tiles are read from the CACHE, where the kernel has put this call's rows
// first (token i in slot i), so earlier chunks of a prompt and this one come through the same map.
template <typename T, int D, int KT, int ROWS = kBulkRows>
constexpr int bulk_smem_bytes() {
  constexpr bool kTma = sizeof(T) == 2;
  return ROWS * D * 4                                        // query rows, fp32
         + 2 * KT * (D * (int)sizeof(T) + (kTma ? 0 : 16))   // two tile stages, storage type, padded rows (or swizzled)
         + KT * bulk_pad_p(ROWS) * 4                         // probabilities of a tile, fp32
         + (sizeof(T) == 2 ? 2 * ROWS * (KT + 8) * 2 : 0)    // bf16 hi and lo parts of the probabilities
         + 64;                                               // mbarriers
}

__device__ __forceinline__ void store_row_part(float* p, const float (&x)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
}
__device__ __forceinline__ void store_row_part(float* p, const float (&x)[2]) {
  *reinterpret_cast<float2*>(p) = make_float2(x[0], x[1]);
}
__device__ __forceinline__ void store_row_part(__nv_bfloat16* p, const float (&x)[4]) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(x[0], x[1]), hi = __floats2bfloat162_rn(x[2], x[3]);
  uint2 t;
  t.x = *reinterpret_cast<const uint32_t*>(&lo);
  t.y = *reinterpret_cast<const uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = t;
}
__device__ __forceinline__ void store_row_part(__nv_bfloat16* p, const float (&x)[2]) {
  *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(x[0], x[1]);
}

// a_i <- a_i + mean over the group's heads of P[t, g, i], one token after the other (the order Algorithm 1 adds them
// in).  Thread tid < KT owns key k0 + tid of the tile; Pt is [key][row] with row = token_in_block * G + head; a_prev is
// the key's score before this block (0 if the key's own token is in the block: it starts from [a, 0]).
template <int G, int KT, int ROWS>
__device__ __forceinline__ void fold_columns(const float* Pt, float* a_l, float a_prev, int k0, int t0, int nk, int n) {
  constexpr int BQ = ROWS / G;
  const int key = k0 + (int)threadIdx.x;
  if ((int)threadIdx.x >= KT || key >= nk) return;
  float a_i = a_prev;
  const float* pr = Pt + threadIdx.x * bulk_pad_p(ROWS);
#pragma unroll
  for (int tok = 0; tok < BQ; ++tok) {
    float pbar = pr[tok * G];
#pragma unroll
    for (int g = 1; g < G; ++g) pbar = __fadd_rn(pbar, pr[tok * G + g]);
    if (G > 1) pbar = __fmul_rn(pbar, 1.0f / (float)G);
    if (key <= t0 + tok && t0 + tok < n) a_i = __fadd_rn(a_i, pbar);
  }
  a_l[key] = a_i;
}

// c[16x8, fp32] += a[16x16, bf16, row-major] . b[16x8, bf16, column-major] on the tensor cores (one warp)
__device__ __forceinline__ void mma_m16n8k16_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Byte offset of element `elem` of key `key` inside a swizzled tile of KT keys (see bulk_smem_bytes).
template <int KT>
__device__ __forceinline__ uint32_t swz_off(int key, int elem) {
  const int chunk = elem >> 3;                           // 16-byte chunk of the row
  return (uint32_t)((chunk >> 3) * (KT * 128) + key * 128 + ((((chunk & 7) ^ (key & 7)) << 4) | ((elem & 7) << 1)));
}

template <typename T, int D, int G, int KT, int ROWS = kBulkRows>
__global__ void __launch_bounds__(bulk_threads(ROWS), ROWS == 32 ? 2 : (KT == 64 ? 4 : 2))
prefill_bulk_kernel(const __grid_constant__ PrefillParams P) {
  constexpr bool kTma = sizeof(T) == 2;          // tiles through the caches' tensor maps
  constexpr int kBulkRows = ROWS;                // (shadows the namespace constants: this instantiation's geometry)
  constexpr int kBulkThreads = bulk_threads(ROWS);
  constexpr int kBulkPadP = bulk_pad_p(ROWS);
  constexpr int BQ = kBulkRows / G;              // tokens per row block
  constexpr int CH = D / 16;                     // channels per partial sum of the reproducible dot
  constexpr int CP = CH / 2;                     // ... as (even, odd) pairs
  constexpr int KPT = KT / 32;                   // keys per thread in the logits phase
  constexpr int RS = D + (kTma ? 0 : 16 / (int)sizeof(T));   // row stride of a tile in elements: 16 bytes of padding, no bank conflicts (kTma: swizzled instead)
  constexpr int ROWB = D * (int)sizeof(T);       // bytes per row
  constexpr int CPT = D / 32;                    // output channels per thread in the P.V phase (fp32 storage)
  constexpr bool kTensorPV = sizeof(T) == 2;     // bf16 storage: P.V on the tensor cores
  constexpr int PS = KT + 8;                     // bf16 row stride of the hi / lo probability tiles
  constexpr int QV = ROWB / 128;                 // 16-byte pieces of the query block per thread
  static_assert(kBulkRows % G == 0 && kBulkThreads == 8 * kBulkRows && KT <= kBulkThreads && kBulkKeys % KT == 0, "thread maps");
  extern __shared__ __align__(1024) unsigned char bulk_smem[];           // (swizzled tiles start on 1024-byte boundaries)
  float* Qs = reinterpret_cast<float*>(bulk_smem);                       // [rows][D] fp32
  T* stage0 = reinterpret_cast<T*>(Qs + kBulkRows * D);                  // 2 x [KT][RS]
  float* Pt = reinterpret_cast<float*>(stage0 + 2 * KT * RS);            // [KT][20]: probabilities, [key][row]
  __nv_bfloat16* Ph = reinterpret_cast<__nv_bfloat16*>(Pt + KT * kBulkPadP);   // [rows][KT + 8] (bf16 storage only)
  __nv_bfloat16* Pl = Ph + kBulkRows * PS;
  uint64_t* full = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(Pt + KT * kBulkPadP) +
                                               (kTensorPV ? 2 * kBulkRows * PS * 2 : 0));

  const int tid = threadIdx.x, w = tid >> 5, ln = tid & 31;
  const int lane_local = blockIdx.x;
  const int b = lane_local / P.n_kv_heads, hk = lane_local % P.n_kv_heads;
  const long long lane = (long long)P.lane0 + lane_local;
  const int Hk = P.n_kv_heads, Hq = Hk * G;
  // The lane may already hold n_old tokens from earlier calls -- uncompressed, so token i sits in slot i with its
  // score a_i so far; the host only sends lanes here whose n_old + n0 cannot exceed the budget.  This call adds n_new
  // tokens (input rows 0 .. n_new-1, global token index n_old + row); n = tokens held afterwards.
  const int n_old = P.lane_state[lane * LS_STRIDE + LS_T];
  const bool consistent = P.lane_state[lane * LS_STRIDE + LS_LEN] == n_old && n_old + P.n0 <= P.s_stride && n_old + P.n0 < P.cap;
  int n_new = P.n0;
  if (P.seq_lens != nullptr) n_new = min(n_new, max(0, P.seq_lens[b % P.batch]));
  const int n = n_old + n_new;
  const T* Qb = reinterpret_cast<const T*>(P.Q) + ((long long)b * P.T_max * Hq + (long long)hk * G) * D;   // + t*Hq*D + g*D
  const T* Kb = reinterpret_cast<const T*>(P.K) + ((long long)b * P.T_max * Hk + hk) * D;                  // + t*Hk*D
  const T* Vb = reinterpret_cast<const T*>(P.V) + ((long long)b * P.T_max * Hk + hk) * D;
  T* Kl = reinterpret_cast<T*>(P.Kc) + lane * (long long)P.cap * D;
  T* Vl = reinterpret_cast<T*>(P.Vc) + lane * (long long)P.cap * D;
  float* a_l = P.a + lane * P.cap;
  float* S = P.S + (long long)lane_local * kBulkRows * P.s_stride;

  // no compression happens in this phase: report "nothing removed" for every token it covers
  if (P.evicted != nullptr)
    for (int t = tid; t < P.n0; t += kBulkThreads) P.evicted[((long long)b * P.T_max + t) * Hk + hk] = -1;
  if (!consistent) {                                     // cannot happen through the library's entry points
    if (tid == 0) atomicOr(P.status, kStatusBadLink);
    return;
  }
  if (n_new == 0) return;

  if (tid == 0) {
    mbar_init(&full[0], kTma ? 1 : KT);                  // every issuing thread arrives once per fill
    mbar_init(&full[1], kTma ? 1 : KT);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // The ring.  Thread r < KT fetches row r of a tile: one bulk copy, counted in bytes on the stage's barrier.  Rows
  // beyond the last key of the block re-fetch that last key (finite values; their probabilities are exactly zero).
  uint32_t parity = 0;                                   // bit s: parity of stage s's next completion
  // (kTma) the tiles are streamed -- every block re-reads them, long after they have left L2 -- while the scratch rows
  // of logits are re-read within the block: the tiles are marked to leave L2 first (measured: 2 to 10 % of the kernel;
  // marking the scratch rows to stay instead made it slower)
  const uint64_t stream_policy = kTma ? l2_policy_evict_first() : 0ull;
  // Keys / values of tokens before n_old come from the cache (slot = token), the others from this call's input.
  auto issue = [&](bool values, int kt, int s, int nk_) {
    if constexpr (kTma) {
      // whole boxes of KT keys out of the cache: keys past nk_ are slots not yet filled (or zero fill past the end of
      // the cache); the causal mask keeps them out of the logits, and the value rows among them are zeroed before they
      // are multiplied
      if (tid == 0) {
        mbar_expect_tx(&full[s], (uint32_t)(KT * ROWB));
#pragma unroll
        for (int h = 0; h < ROWB / 128; ++h)
          tensor_g2s_2d_hint(reinterpret_cast<unsigned char*>(stage0) + (size_t)s * KT * ROWB + h * KT * 128, values ? P.vmap : P.kmap,
                             h * 64, (int)(lane * P.cap) + kt * KT, &full[s], stream_policy);
      }
    } else if (tid < KT) {
      const int r = min(kt * KT + tid, nk_ - 1);
      const T* src = r < n_old ? (values ? Vl : Kl) + (long long)r * D : (values ? Vb : Kb) + (long long)(r - n_old) * Hk * D;
      mbar_expect_tx(&full[s], ROWB);
      bulk_g2s(stage0 + (s * KT + tid) * RS, src, ROWB, &full[s]);
    }
  };
  constexpr bool kKeys = false, kValues = true;
  auto wait_stage = [&](int s) {
    mbar_wait(&full[s], (parity >> s) & 1u, P.status);
    parity ^= 1u << s;
  };
  // query rows of a block as 16-byte pieces in registers: piece c -> row c / (ROWB/16); row = token_in_block * G + head
  uint4 qpre[QV];
  auto load_q = [&](int t0_) {
#pragma unroll
    for (int i = 0; i < QV; ++i) {
      const int c = tid + kBulkThreads * i;
      const int r = c / (ROWB / 16), q = c % (ROWB / 16);
      const int tok = t0_ + r / G, g = r % G;
      qpre[i] = make_uint4(0u, 0u, 0u, 0u);
      if (tok < n) qpre[i] = reinterpret_cast<const uint4*>(Qb + ((long long)(tok - n_old) * Hq + g) * D)[q];
    }
  };
  auto store_q = [&]() {
#pragma unroll
    for (int i = 0; i < QV; ++i) {
      const int c = tid + kBulkThreads * i;
      const int r = c / (ROWB / 16), q = c % (ROWB / 16);
      if constexpr (sizeof(T) == 2) {
        float* d = Qs + r * D + q * 8;
        const uint4 t = qpre[i];
        *reinterpret_cast<float4*>(d) = make_float4(__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xffff0000u),
                                                    __uint_as_float(t.y << 16), __uint_as_float(t.y & 0xffff0000u));
        *reinterpret_cast<float4*>(d + 4) = make_float4(__uint_as_float(t.z << 16), __uint_as_float(t.z & 0xffff0000u),
                                                        __uint_as_float(t.w << 16), __uint_as_float(t.w & 0xffff0000u));
      } else {
        *reinterpret_cast<uint4*>(Qs + r * D + q * 4) = qpre[i];
      }
    }
  };
  load_q(n_old);
  if constexpr (!kTma) {
    issue(kKeys, 0, 0, min(n_old + BQ, n));
    if (min(n_old + BQ, n) > KT) issue(kKeys, 1, 1, min(n_old + BQ, n));
  }

  // the cache after n uncompressed steps: token i in slot i, linked in order (Algorithm 1 appends, nothing is removed)
  {
    constexpr int Q8 = ROWB / 16;                        // 16-byte pieces per row
    for (int c = tid; c < n_new * Q8; c += kBulkThreads) {
      const int r = c / Q8, q = c % Q8;
      reinterpret_cast<uint4*>(Kl + (long long)(n_old + r) * D)[q] = reinterpret_cast<const uint4*>(Kb + (long long)r * Hk * D)[q];
      reinterpret_cast<uint4*>(Vl + (long long)(n_old + r) * D)[q] = reinterpret_cast<const uint4*>(Vb + (long long)r * Hk * D)[q];
    }
    int32_t* pos_l = P.pos + lane * P.cap;
    int32_t* next_l = P.next + lane * P.cap;
    int32_t* prev_l = P.prev + lane * P.cap;
    for (int i = n_old + tid; i < n; i += kBulkThreads) {
      pos_l[i] = i;
      next_l[i] = i + 1 < n ? i + 1 : -1;
      prev_l[i] = i - 1;
    }
    if (tid == 0) {
      if (n_old > 0) next_l[n_old - 1] = n_old;          // the old tail gets a right neighbour
      int32_t* st = P.lane_state + lane * LS_STRIDE;
      st[LS_LEN] = n;
      st[LS_T] = n;
      st[LS_HEAD] = 0;
      st[LS_TAIL] = n - 1;
      st[LS_FREE] = n;                                   // while growing, slots fill in arrival order
    }
  }
  if constexpr (kTma) {
    // the tiles come out of the cache rows just written: make those writes visible to the copy engine first
    asm volatile("fence.proxy.async.global;" ::: "memory");
    __syncthreads();
    issue(kKeys, 0, 0, min(n_old + BQ, n));
    if (min(n_old + BQ, n) > KT) issue(kKeys, 1, 1, min(n_old + BQ, n));
  }

  for (int t0 = n_old; t0 < n; t0 += BQ) {
    const int nk = min(t0 + BQ, n);                      // keys 0 .. nk-1 are visible to some row of the block
    const int n_tiles = (nk + KT - 1) / KT;
    int t_row[4];                                        // token of each of my 4 rows
    bool act[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      t_row[i] = t0 + (4 * w + i) / G;
      act[i] = t_row[i] < n;
    }
    store_q();                                           // (the previous block's last barrier freed Qs)
    __syncthreads();
    if (t0 + BQ < n) load_q(t0 + BQ);                    // next block's queries: in flight during this whole block

    // ---- phase 1: logits of the row block, tile by tile (K tiles 0 and 1 are already in flight) -------------------
    float row_max[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
    for (int kt = 0; kt < n_tiles; ++kt) {
      const int k0 = kt * KT, s = kt & 1;
      wait_stage(s);
      const T* Kt = stage0 + s * KT * RS;
      // The reproducible dot: 16 partial sums over blocks of D/16 channels (even- and odd-channel fma chains, added),
      // combined as the butterfly p_r + p_{r xor off}, off = 8, 4, 2, 1.  The blocks are visited in the order that
      // lets the butterfly's additions be done as soon as both operands exist (a fixed tree; fp addition commutes).
      float st1[4 * KPT], st2[4 * KPT], st3[4 * KPT], st4[4 * KPT], dot[4 * KPT];
#pragma unroll
      for (int sb = 0; sb < 16; ++sb) {
        const int blk = ((sb & 1) << 3) | ((sb & 2) << 1) | ((sb & 4) >> 1) | ((sb & 8) >> 3);   // 0,8,4,12,2,10,6,14,1,...
        f32x2 qv[4][CP], kv[KPT][CP];
#pragma unroll
        for (int i = 0; i < 4; ++i) load_pairs<CP>(Qs + (4 * w + i) * D + blk * CH, qv[i]);
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
          if constexpr (kTma)
            load_pairs<CP>(reinterpret_cast<const T*>(reinterpret_cast<const unsigned char*>(Kt) + swz_off<KT>(ln + 32 * j, blk * CH)), kv[j]);
          else
            load_pairs<CP>(Kt + (ln + 32 * j) * RS + blk * CH, kv[j]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
#pragma unroll
          for (int j = 0; j < KPT; ++j) {
            const int o = i * KPT + j;
            f32x2 acc = 0ull;
#pragma unroll
            for (int e = 0; e < CP; ++e) acc = fma2(qv[i][e], kv[j][e], acc);
            float v = __fadd_rn(lo_of(acc), hi_of(acc));
            if (sb & 1) {
              v = __fadd_rn(st1[o], v);
              if (sb & 2) {
                v = __fadd_rn(st2[o], v);
                if (sb & 4) {
                  v = __fadd_rn(st3[o], v);
                  if (sb & 8) dot[o] = __fadd_rn(st4[o], v);
                  else st4[o] = v;
                } else st3[o] = v;
              } else st2[o] = v;
            } else st1[o] = v;
          }
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
          const int key = k0 + ln + 32 * j;
          const bool ok = act[i] && key <= t_row[i];     // causal: the row's own token is its last key
          const float sc = ok ? __fmul_rn(P.scale, dot[i * KPT + j]) : -INFINITY;
          S[(long long)(4 * w + i) * P.s_stride + key] = sc;
          row_max[i] = fmaxf(row_max[i], sc);
        }
      }
      __syncthreads();                                   // everybody is done with the stage
      if (kt + 2 < n_tiles) issue(kKeys, kt + 2, s, nk);
    }
    // both stages are free: put the first V tiles in flight, they land while the exponentials are computed
    issue(kValues, 0, 0, nk);
    if (n_tiles > 1) issue(kValues, 1, 1, nk);
    // ---- phase 2: exponentials in place and the integer-sum normaliser (each thread re-reads what it wrote) ------
    float Z[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float m = row_max[i];
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
      unsigned long long z = 0ull;
      float* Srow = S + (long long)(4 * w + i) * P.s_stride;
#pragma unroll 4
      for (int key = ln; key < n_tiles * KT; key += 32) {
        const float sc = Srow[key];
        const float e = (act[i] && sc != -INFINITY) ? repro_exp(__fsub_rn(sc, m)) : 0.f;
        Srow[key] = e;
        z += __float2ull_rz(__fmul_rn(e, 1099511627776.0f));
      }
      z = warp_sum_u64(z);
      Z[i] = __fmul_rn(__ull2float_rn(z), 1.0f / 1099511627776.0f);
    }
    // ---- phase 3: probabilities, score accumulation, outputs -----------------------------------------------------
    constexpr int NTW = D / 32;                          // tensor path: 8-channel n-tiles per warp
    float cacc[kTensorPV ? NTW : 1][4];
    f32x2 o_acc[kTensorPV ? 1 : 4][kTensorPV ? 1 : CPT / 2];
    if constexpr (kTensorPV) {
#pragma unroll
      for (int nt = 0; nt < NTW; ++nt) cacc[nt][0] = cacc[nt][1] = cacc[nt][2] = cacc[nt][3] = 0.f;
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int c = 0; c < CPT / 2; ++c) o_acc[i][c] = 0ull;
    }
    for (int kt = 0; kt < n_tiles; ++kt) {
      const int k0 = kt * KT, s = kt & 1;
      const int my_key = k0 + tid;
      const float a_prev = (tid < KT && my_key < nk && my_key < t0) ? a_l[my_key] : 0.f;
      // all of the tile's exponentials first: the IEEE division below may call its slow path, and a call keeps the
      // compiler from moving later loads ahead of it (one L2 round trip per value instead of one per tile)
      float ev[KPT][4];
#pragma unroll
      for (int j = 0; j < KPT; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) ev[j][i] = S[(long long)(4 * w + i) * P.s_stride + k0 + ln + 32 * j];
#pragma unroll
      for (int j = 0; j < KPT; ++j) {
        const int kk = ln + 32 * j;
        float p[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          p[i] = act[i] ? __fdiv_rn(ev[j][i], Z[i]) : 0.f;
          if constexpr (kTensorPV) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(p[i]);
            Ph[(4 * w + i) * PS + kk] = hi;
            Pl[(4 * w + i) * PS + kk] = __float2bfloat16_rn(p[i] - __bfloat162float(hi));
          }
        }
        *reinterpret_cast<float4*>(Pt + kk * kBulkPadP + 4 * w) = make_float4(p[0], p[1], p[2], p[3]);
      }
      wait_stage(s);                                     // the V tile
      T* Vt = stage0 + s * KT * RS;
      if constexpr (kTma) {
        if (k0 + KT > nk) {
          // rows past the block's last key are not this block's: zero them (0 * NaN would reach the accumulators)
          const int r0 = nk - k0;
          for (int idx = tid; idx < (KT - r0) * (ROWB / 16); idx += kBulkThreads) {
            const int row = r0 + idx / (ROWB / 16), c16 = idx % (ROWB / 16);
            *reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(Vt) + (c16 >> 3) * (KT * 128) + row * 128 + (c16 & 7) * 16) =
                make_uint4(0u, 0u, 0u, 0u);
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // before the stage is refilled
        }
      }
      __syncthreads();                                   // the probability tiles (and the zeroed rows)
      fold_columns<G, KT, ROWS>(Pt, a_l, a_prev, k0, t0, nk, n);
      if constexpr (kTensorPV) {
        // O += P . V on the tensor cores (the outputs are not part of the reproducible chain).  Warp w takes all 16
        // rows and channels [w*D/4, (w+1)*D/4).  Fragment addresses: A (P, row-major [row][key]): thread i -> row
        // (i%8) + 8*((i/8)&1), key 8*(i/16); B (V, [key][channel], read transposed): thread i -> key (i%8) +
        // 8*((i/8)&1), channel 8*(i/16).
        // (blocks of 32 rows: warps 4 .. 7 do the same for rows 16 .. 31)
        const int ksteps = (min(KT, nk - k0) + 15) / 16;
        const int wq = w & 3, wr = (w >> 2) * 16;        // the warp's channel quarter and first row
        const int frow = (ln & 7) + ((ln >> 3) & 1) * 8, fcol = (ln >> 4) * 8;
        const uint32_t a_off = (uint32_t)(((wr + frow) * PS + fcol) * 2);
        const uint32_t ph_base = smem_u32(Ph) + a_off, pl_base = smem_u32(Pl) + a_off;
        const uint32_t v_base = smem_u32(Vt) + (uint32_t)((frow * RS + wq * (D / 4) + fcol) * 2);   // (padded rows)
        for (int ks = 0; ks < ksteps; ++ks) {
          uint32_t ah[4], al[4];
          asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                       : "=r"(ah[0]), "=r"(ah[1]), "=r"(ah[2]), "=r"(ah[3]) : "r"(ph_base + ks * 32) : "memory");
          asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                       : "=r"(al[0]), "=r"(al[1]), "=r"(al[2]), "=r"(al[3]) : "r"(pl_base + ks * 32) : "memory");
#pragma unroll
          for (int np = 0; np < NTW / 2; ++np) {
            uint32_t bf[4];
            const uint32_t v_addr = kTma ? smem_u32(Vt) + swz_off<KT>(ks * 16 + frow, wq * (D / 4) + fcol + np * 16)
                                         : v_base + (uint32_t)(ks * 16 * RS * 2 + np * 32);
            asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                         : "=r"(bf[0]), "=r"(bf[1]), "=r"(bf[2]), "=r"(bf[3])
                         : "r"(v_addr) : "memory");
            mma_m16n8k16_bf16(cacc[2 * np], ah, bf[0], bf[1]);
            mma_m16n8k16_bf16(cacc[2 * np], al, bf[0], bf[1]);
            mma_m16n8k16_bf16(cacc[2 * np + 1], ah, bf[2], bf[3]);
            mma_m16n8k16_bf16(cacc[2 * np + 1], al, bf[2], bf[3]);
          }
        }
      } else {
        // fp32 storage: packed fp32 FMAs; warp w keeps its 4 rows, each thread CPT channels
        // the tile's products are summed on their own and then added to the running output: thousands of keys in one
        // sequential fp32 chain would cost more accuracy than the 1e-5 output tolerance leaves
        f32x2 o_tile[4][CPT / 2];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int c = 0; c < CPT / 2; ++c) o_tile[i][c] = 0ull;
        const int kmax = min(KT, nk - k0);
        for (int kk = 0; kk < kmax; ++kk) {
          const float4 p4 = *reinterpret_cast<const float4*>(Pt + kk * kBulkPadP + 4 * w);
          const f32x2 pp[4] = {pack2(p4.x, p4.x), pack2(p4.y, p4.y), pack2(p4.z, p4.z), pack2(p4.w, p4.w)};
          f32x2 vv[CPT / 2];
          const float* vrow = reinterpret_cast<const float*>(Vt) + kk * RS + ln * CPT;
          if constexpr (CPT == 4) {
            load_pairs<2>(vrow, vv);
          } else {
            const float2 t = *reinterpret_cast<const float2*>(vrow);
            vv[0] = pack2(t.x, t.y);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int c = 0; c < CPT / 2; ++c) o_tile[i][c] = fma2(pp[i], vv[c], o_tile[i][c]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int c = 0; c < CPT / 2; ++c)
            o_acc[i][c] = pack2(lo_of(o_acc[i][c]) + lo_of(o_tile[i][c]), hi_of(o_acc[i][c]) + hi_of(o_tile[i][c]));
      }
      __syncthreads();                                   // everybody is done with the stage and the probability tiles
      if (kt + 2 < n_tiles) issue(kValues, kt + 2, s, nk);
    }
    // both stages are free again: the next block's first K tiles travel while this block's outputs are stored
    if (t0 + BQ < n) {
      const int nk_next = min(t0 + 2 * BQ, n);
      issue(kKeys, 0, 0, nk_next);
      if (nk_next > KT) issue(kKeys, 1, 1, nk_next);
    }
    if (P.out != nullptr) {
      if constexpr (kTensorPV) {
        // accumulator fragment: rows ln/4 and ln/4 + 8, channels (ln%4)*2, +1 of each n-tile
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int rho = (w >> 2) * 16 + (ln >> 2) + 8 * h;
          const int t = t0 + rho / G, g = rho % G;
          if (t >= n) continue;
          T* dst = reinterpret_cast<T*>(P.out) + (((long long)b * P.T_max + (t - n_old)) * Hq + (long long)hk * G + g) * D + (w & 3) * (D / 4) + (ln & 3) * 2;
#pragma unroll
          for (int nt = 0; nt < NTW; ++nt) {
            const float x[2] = {cacc[nt][2 * h], cacc[nt][2 * h + 1]};
            store_row_part(dst + nt * 8, x);
          }
        }
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (!act[i]) continue;
          const int g = (4 * w + i) % G;
          T* dst = reinterpret_cast<T*>(P.out) + (((long long)b * P.T_max + (t_row[i] - n_old)) * Hq + (long long)hk * G + g) * D + ln * CPT;
          float x[CPT];
#pragma unroll
          for (int c = 0; c < CPT / 2; ++c) { x[2 * c] = lo_of(o_acc[i][c]); x[2 * c + 1] = hi_of(o_acc[i][c]); }
          store_row_part(dst, x);
        }
      }
    }
  }
}

}  // namespace wkv
