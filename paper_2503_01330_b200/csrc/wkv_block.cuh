// Blocked prompt tail of WeightedKV (Algorithm 1) for sm_100a.
//
// Algorithm 1 streams a prompt: every token is one pass over the lane's cache.  Once a lane is full every token also
// removes an entry, so the tokens of a prompt cannot be treated as one dense problem any more -- but the cache changes
// by only one row per token.  For a block of B consecutive tokens this file reads the cache twice instead of 2B times:
//
//   block_logits_kernel   one sweep over the K rows as they are before the block: the logits of all B tokens' queries
//                         against every slot (reproducible dot, parked per token), plus the B x B logits of the block's
//                         tokens against the block's own keys.
//   lane_epilogue_block_kernel  one launch (wkv_kernels.cuh, StepParams::block_tokens > 0): per lane, token after token,
//                         exactly the per-token epilogue of the streamed step -- probabilities, score fold, pick, merge,
//                         relink -- on the parked logits of each token.  An entry that joined inside the block is
//                         recognised by its position and takes its logit from the B x B table; removed entries are gone
//                         from the chain as in streaming.  Each step writes its token's rows into the freed slot, leaves
//                         the token's probabilities in a table (slot order) and records every value row that it changes
//                         as it was before.  (lane_epilogue_kernel does one such step per launch when given block_step.)
//   block_pv_kernel       one sweep over the V rows as they are after the block: sum_s P[token][s] * V[s] for all B tokens.
//   block_out_kernel      per query row of the block: adds the units' partial sums and, for every recorded change,
//                         P[token][s] * (row as it was when the token attended - row as it is now) for the tokens in
//                         front of the change: the attention output uses V before the step's own merge, as in Algorithm 1.
//
// Everything that decides a removal (logits, probabilities, accumulated scores, pick, merged values) is computed by the
// same code as in the streamed step, in the same order, so the state after the block is bit-identical; the outputs
// agree within the output tolerance.  Requirement: window > B, so that an entry removed inside the block, and its right
// neighbour, are never tokens of the block itself.
#pragma once
#include "wkv_kernels.cuh"

namespace wkv {

struct BlockParams {
  void* Kc;                  // cache, as in StepParams
  void* Vc;
  int32_t* lane_state;
  const void* Q;             // prompt tensors of the call: [batch, T_max, heads, D]
  const void* K;
  void* out;                 // [batch, T_max, n_q_heads, D] or nullptr
  const int32_t* seq_lens;   // [batch] or nullptr
  float* logits;             // [lanes][rows][cap]  rows = block_tokens * G
  float* lgx;                // [lanes][rows][block_tokens]
  const float* ptab;         // [lanes][rows][cap] probabilities in slot order (+ one tile of padding at the very end)
  float* opart;              // [lanes][n_units][rows][D] partial sums of the value sweep
  const float* rec_rows;     // [lanes][2 * block_tokens][D]
  const int32_t* rec_slot;   // [lanes][2 * block_tokens]
  uint32_t* status;
  long long q_bs, kv_bs, out_bs;   // batch strides in elements
  long long q_ts, kv_ts, out_ts;   // token strides in elements
  int lane0, n_kv_heads, cap, budget;
  int tok0;                  // index of the block's first token inside the call
  int n_tok;                 // tokens of this block (<= block_tokens)
  int block_tokens;          // B
  int group;                 // query heads per kv head
  int n_units;               // CTAs per lane in the two sweeps
  float scale;
  // Tensor map over the value cache (as in StepParams), for the value sweep on the tensor cores.
  alignas(64) unsigned char vmap[128];
};

// tokens of the block that sequence b still has (ragged prompts end inside a block)
__device__ __forceinline__ int block_active_tokens(const BlockParams& P, int b) {
  if (P.seq_lens == nullptr) return P.n_tok;
  return max(0, min(P.n_tok, P.seq_lens[b] - P.tok0));
}

// Shared memory of the two sweeps: a ring of single tiles | an extra tile (the block's own keys) or the tile's
// probabilities per stage | warp partials | mbarriers.
template <typename T, int D, int R>
struct BlockCfg {
  static constexpr int kRowBytes = D * (int)sizeof(T);
  static constexpr int kTileBytes = kTileSlots * kRowBytes;
  static constexpr int kStages = 4;
  static constexpr int kProbBytes = R * kTileSlots * 4;                      // [R][32] fp32 per stage (value sweep)
  static constexpr int kLogitsSmem = kStages * kTileBytes + kTileBytes + 2 * kStages * 8 + 64;
  // Value sweep on the tensor cores: bf16 rows, R = 8 tokens (the n dimension of mma.m16n8k8), and a tensor map for
  // the swizzled V tiles (a stage must then start on a 1024-byte boundary, which kTileBytes + kProbBytes keeps).
  static constexpr bool kPvMma = sizeof(T) == 2 && R == 8 && D % 64 == 0;
  static constexpr int kVHalves = kRowBytes / 128;
  static constexpr int kVHalfBytes = kTileSlots * 128;
  static constexpr int kPvSmem = kStages * (kTileBytes + kProbBytes) + kConsumerWarps * R * D * 4 + 2 * kStages * 8 + 64;
};

// ------------------------------------------------------------------------------------------------
// sweep 1: logits of R = block_tokens * group query rows against the lane's K rows
// ------------------------------------------------------------------------------------------------
template <typename T, int D, int R>
__global__ void __launch_bounds__(kThreads) block_logits_kernel(const BlockParams P) {
  using BC = BlockCfg<T, D, R>;
  using SC = Scanner<T, D, R>;
  constexpr int NS = BC::kStages;
  constexpr int NC = kConsumerWarps * 32;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* ring = smem_raw;
  T* own = reinterpret_cast<T*>(ring + NS * BC::kTileBytes);                 // the block's own keys as one tile
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(ring + (NS + 1) * BC::kTileBytes);
  uint64_t* empty_bar = full_bar + NS;
  const int tid = threadIdx.x, warp = tid >> 5, lane_id = tid & 31;
  const int unit = blockIdx.x % P.n_units;
  const int lane_local = blockIdx.x / P.n_units;
  const int b = lane_local / P.n_kv_heads, hk = lane_local % P.n_kv_heads;
  const int n_act = block_active_tokens(P, b);
  if (n_act == 0) return;
  const long long lane = (long long)P.lane0 + lane_local;
  const int* st = P.lane_state + lane * LS_STRIDE;
  const int len0 = st[LS_LEN];
  // slots that hold an entry at some step of the block: the lane's entries now, plus the slots its growth takes
  const int L = min(len0 + n_act, P.budget + 1);
  const T* Kl = reinterpret_cast<const T*>(P.Kc) + lane * (long long)P.cap * D;
  const int tiles_total = (L + kTileSlots - 1) / kTileSlots;
  const int base = tiles_total / P.n_units, extra = tiles_total % P.n_units;
  const int tile_begin = unit * base + min(unit, extra);
  const int n_tiles = base + (unit < extra ? 1 : 0);
  if (warp == kConsumerWarps) {
    if (lane_id == 0) {
      for (int s = 0; s < NS; ++s) {
        mbar_init(&full_bar[s], 1);
        mbar_init(&empty_bar[s], kConsumerWarps);
      }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    asm volatile("bar.arrive 2, %0;" ::"n"(kThreads) : "memory");
    if (lane_id == 0) {
      for (int i = 0; i < n_tiles; ++i) {
        const int s = i % NS;
        if (i >= NS) mbar_wait(&empty_bar[s], ((i / NS) - 1) & 1, P.status);
        const int slot0 = (tile_begin + i) * kTileSlots;
        const uint32_t bytes = (uint32_t)min(kTileSlots, L - slot0) * BC::kRowBytes;
        mbar_expect_tx(&full_bar[s], bytes);
        bulk_g2s_hint(ring + (size_t)s * BC::kTileBytes, Kl + (long long)slot0 * D, bytes, &full_bar[s], l2_policy_evict_first());   // streamed once
      }
    }
    return;
  }
  // query rows: row r = token r / group, head r % group; tokens past the sequence's end repeat its last token (unused)
  SC sc;
  {
    const T* Qb = reinterpret_cast<const T*>(P.Q) + b * P.q_bs + (long long)P.tok0 * P.q_ts + (long long)hk * P.group * D;
    sc.begin_rows(Qb, P.q_ts, P.group, n_act);
  }
  // the block's own keys, as the first rows of a tile of their own (unit 0 only)
  if (unit == 0) {
    const T* Kb = reinterpret_cast<const T*>(P.K) + b * P.kv_bs + (long long)P.tok0 * P.kv_ts + (long long)hk * D;
    for (int idx = tid; idx < kTileSlots * D; idx += NC) {
      const int r = idx / D, c = idx % D;
      own[idx] = r < n_act ? Kb[(long long)r * P.kv_ts + c] : from_f32<T>(0.f);
    }
  }
  asm volatile("bar.sync 2, %0;" ::"n"(kThreads) : "memory");                // barriers exist, own keys written
  float* lg = P.logits + (long long)lane_local * R * P.cap;
  for (int i = 0; i < n_tiles; ++i) {
    const int s = i % NS;
    mbar_wait(&full_bar[s], (i / NS) & 1, P.status);
    const T* tK = reinterpret_cast<const T*>(ring + (size_t)s * BC::kTileBytes);
    const int slot0 = (tile_begin + i) * kTileSlots;
    float sv[SC::PASSES];
    bool valid[SC::PASSES];
    sc.logits(tK, slot0, L, P.scale, sv, valid);
    SC::park(sv, slot0, L, lg, P.cap, 0);
    release_stage(&empty_bar[s]);
  }
  if (unit == 0) {
    float sv[SC::PASSES];
    bool valid[SC::PASSES];
    sc.logits(own, 0, n_act, P.scale, sv, valid);
    SC::park(sv, 0, n_act, P.lgx + (long long)lane_local * R * P.block_tokens, P.block_tokens, 0);
  }
}

// ------------------------------------------------------------------------------------------------
// sweep 2: sum_s P[row][s] * V[s] over the unit's slots, all R rows at once
// ------------------------------------------------------------------------------------------------
template <typename T, int D, int R, bool kMma>
__global__ void __launch_bounds__(kThreads) block_pv_kernel(const __grid_constant__ BlockParams P) {
  using BC = BlockCfg<T, D, R>;
  static_assert(!kMma || BC::kPvMma, "the tensor-core sweep needs bf16 rows and blocks of 8 query rows");
  constexpr int NS = BC::kStages;
  constexpr int NC = kConsumerWarps * 32;
  constexpr int LPR = 16, CH = D / 16, CP = CH / 2, RPP = 32 / LPR, PASSES = 8 / RPP;
  constexpr int kStage = BC::kTileBytes + BC::kProbBytes;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* ring = smem_raw;
  float* warp_part = reinterpret_cast<float*>(ring + NS * kStage);           // [warp][R][D]
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(warp_part + kConsumerWarps * R * D);
  uint64_t* empty_bar = full_bar + NS;
  const int tid = threadIdx.x, warp = tid >> 5, lane_id = tid & 31;
  const int unit = blockIdx.x % P.n_units;
  const int lane_local = blockIdx.x / P.n_units;
  const int b = lane_local / P.n_kv_heads;
  if (block_active_tokens(P, b) == 0) return;
  const long long lane = (long long)P.lane0 + lane_local;
  const int* st = P.lane_state + lane * LS_STRIDE;
  // slots that have ever held an entry: all of them once the lane has compressed, else the entries it holds
  const int L = st[LS_T] > P.budget ? P.budget + 1 : st[LS_LEN];
  const T* Vl = reinterpret_cast<const T*>(P.Vc) + lane * (long long)P.cap * D;
  const float* pt = P.ptab + (long long)lane_local * R * P.cap;
  const int tiles_total = (L + kTileSlots - 1) / kTileSlots;
  const int base = tiles_total / P.n_units, extra = tiles_total % P.n_units;
  const int tile_begin = unit * base + min(unit, extra);
  const int n_tiles = base + (unit < extra ? 1 : 0);
  if (tid == NC) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], kConsumerWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (warp == kConsumerWarps) {
    if (lane_id == 0) {
      for (int i = 0; i < n_tiles; ++i) {
        const int s = i % NS;
        if (i >= NS) mbar_wait(&empty_bar[s], ((i / NS) - 1) & 1, P.status);
        const int slot0 = (tile_begin + i) * kTileSlots;
        const uint32_t bytes = (uint32_t)min(kTileSlots, L - slot0) * BC::kRowBytes;
        unsigned char* dst = ring + (size_t)s * kStage;
        if constexpr (kMma) {
          // whole boxes of 32 rows in the swizzled layout (rows past the lane's slots: other bytes, zeroed by the consumers)
          mbar_expect_tx(&full_bar[s], (uint32_t)(BC::kVHalves * BC::kVHalfBytes + BC::kProbBytes));
#pragma unroll
          for (int h = 0; h < BC::kVHalves; ++h)
            tensor_g2s_2d_hint(dst + h * BC::kVHalfBytes, P.vmap, h * 64, (int)(lane * P.cap) + slot0, &full_bar[s], l2_policy_evict_first());
        } else {
          mbar_expect_tx(&full_bar[s], bytes + (uint32_t)BC::kProbBytes);
          bulk_g2s_hint(dst, Vl + (long long)slot0 * D, bytes, &full_bar[s], l2_policy_evict_first());
        }
        // the tile's probabilities: 32 slots of every row (entries past the lane's slots are never used)
        for (int r = 0; r < R; ++r)
          bulk_g2s(dst + BC::kTileBytes + r * kTileSlots * 4, pt + (long long)r * P.cap + slot0, kTileSlots * 4, &full_bar[s]);
      }
    }
  } else if constexpr (kMma) {
    // (V rows)^T [channels x 8 rows] times the block's probabilities [8 rows x R tokens] per warp and tile, in blocks of
    // 16 channels: mma.m16n8k8 with the value fragments read transposed out of the swizzled tile, each probability as a
    // bf16 high part plus a bf16 low part (two products into one accumulator).  Warp w owns rows 8w .. 8w+7 of every
    // tile.  Accumulator of block j: channels 16j + c and 16j + 8 + c (c = lane / 4) of tokens 2q and 2q+1 (q = lane % 4).
    using SW = Scanner<T, D, 4>;                         // its v_word() addresses the swizzled tile
    constexpr int NB = D / 16;
    float oc[NB][4];
#pragma unroll
    for (int j = 0; j < NB; ++j) oc[j][0] = oc[j][1] = oc[j][2] = oc[j][3] = 0.f;
    const int tokn = lane_id >> 2, q2 = (lane_id & 3) * 2;                // B fragment: column (token), first of its two rows
    for (int i = 0; i < n_tiles; ++i) {
      const int s = i % NS;
      mbar_wait(&full_bar[s], (i / NS) & 1, P.status);
      T* tV = reinterpret_cast<T*>(ring + (size_t)s * kStage);
      const float* tP = reinterpret_cast<const float*>(ring + (size_t)s * kStage + BC::kTileBytes);
      const int slot0 = (tile_begin + i) * kTileSlots;
      if (slot0 + kTileSlots > L) {
        // ragged tile: rows beyond L hold other bytes, possibly NaN patterns, and 0 * NaN would reach the accumulators
        for (int w = lane_id; w < 8 * (BC::kRowBytes / 4); w += 32) {
          const int r = w / (BC::kRowBytes / 4);
          if (slot0 + warp * 8 + r >= L) *SW::v_word(tV, warp * 8 + r, w % (BC::kRowBytes / 4)) = 0u;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // before the stage is refilled
        __syncwarp();
      }
      const int row = warp * 8 + q2;
      float2 p = *reinterpret_cast<const float2*>(tP + tokn * kTileSlots + row);
      if (slot0 + row >= L) p.x = 0.f;                                    // entries past the lane's slots are stale
      if (slot0 + row + 1 >= L) p.y = 0.f;
      const __nv_bfloat162 hi = __floats2bfloat162_rn(p.x, p.y);
      const float2 hf = __bfloat1622float2(hi);
      const __nv_bfloat162 lo = __floats2bfloat162_rn(p.x - hf.x, p.y - hf.y);
      const uint32_t bh = *reinterpret_cast<const uint32_t*>(&hi), bl = *reinterpret_cast<const uint32_t*>(&lo);
#pragma unroll
      for (int jj = 0; jj < NB / 2; ++jj) {
        uint32_t af[4];
        ldmatrix_x4_trans(af, SW::v_word(tV, warp * 8 + (lane_id & 7), (4 * jj + (lane_id >> 3)) * 4));
        mma_m16n8k8_bf16(oc[2 * jj], af[0], af[1], bh);
        mma_m16n8k8_bf16(oc[2 * jj], af[0], af[1], bl);
        mma_m16n8k8_bf16(oc[2 * jj + 1], af[2], af[3], bh);
        mma_m16n8k8_bf16(oc[2 * jj + 1], af[2], af[3], bl);
      }
      release_stage(&empty_bar[s]);
    }
    {
      const int c = lane_id >> 2;
      float* wa = warp_part + (warp * R + q2) * D;       // token 2q
      float* wb = wa + D;                                // token 2q + 1
#pragma unroll
      for (int j = 0; j < NB; ++j) {
        wa[16 * j + c] = oc[j][0];
        wb[16 * j + c] = oc[j][1];
        wa[16 * j + 8 + c] = oc[j][2];
        wb[16 * j + 8 + c] = oc[j][3];
      }
    }
  } else {
    const int rg = lane_id / LPR, l = lane_id % LPR;
    f32x2 acc[R][CP];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int e = 0; e < CP; ++e) acc[r][e] = 0ull;
    for (int i = 0; i < n_tiles; ++i) {
      const int s = i % NS;
      mbar_wait(&full_bar[s], (i / NS) & 1, P.status);
      const T* tV = reinterpret_cast<const T*>(ring + (size_t)s * kStage);
      const float* tP = reinterpret_cast<const float*>(ring + (size_t)s * kStage + BC::kTileBytes);
      const int slot0 = (tile_begin + i) * kTileSlots;
#pragma unroll
      for (int ps = 0; ps < PASSES; ++ps) {
        const int row = warp * 8 + ps * RPP + rg;
        if (slot0 + row < L) {                                           // rows beyond hold stale bytes, possibly NaN
          f32x2 vf[CP];
          load_pairs<CP>(tV + row * D + l * CH, vf);
#pragma unroll
          for (int r = 0; r < R; ++r) {
            const float p = tP[r * kTileSlots + row];
            const f32x2 p2 = pack2(p, p);
#pragma unroll
            for (int e = 0; e < CP; ++e) acc[r][e] = fma2(p2, vf[e], acc[r][e]);
          }
        }
      }
      release_stage(&empty_bar[s]);
    }
    // the warp's two row groups, then the warp's partial to shared memory
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int e = 0; e < CP; ++e) {
        const f32x2 o = __shfl_xor_sync(0xffffffffu, acc[r][e], 16);
        acc[r][e] = pack2(lo_of(acc[r][e]) + lo_of(o), hi_of(acc[r][e]) + hi_of(o));
      }
    if (rg == 0) {
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int e = 0; e < CP; ++e) {
          warp_part[(warp * R + r) * D + l * CH + 2 * e] = lo_of(acc[r][e]);
          warp_part[(warp * R + r) * D + l * CH + 2 * e + 1] = hi_of(acc[r][e]);
        }
    }
  }
  __syncthreads();
  float* dst = P.opart + ((long long)lane_local * P.n_units + unit) * R * D;
  for (int idx = tid; idx < R * D; idx += kThreads) {
    float o = 0.f;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; ++w) o += warp_part[w * R * D + idx];
    dst[idx] = o;
  }
}

// ------------------------------------------------------------------------------------------------
// outputs of the block's tokens: partial sums of the units + what the rows changed inside the block contributed before
// they changed
// ------------------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(D) block_out_kernel(const BlockParams P) {
  // one CTA per (lane, query row of the block), one thread per channel
  const int c = threadIdx.x;
  const int R = P.block_tokens * P.group;
  const int lane_local = blockIdx.x / R, row = blockIdx.x % R;
  const int tok = row / P.group, g = row % P.group;
  const int b = lane_local / P.n_kv_heads, hk = lane_local % P.n_kv_heads;
  const int n_act = block_active_tokens(P, b);
  if (tok >= n_act || P.out == nullptr) return;
  const long long lane = (long long)P.lane0 + lane_local;
  const T* Vl = reinterpret_cast<const T*>(P.Vc) + lane * (long long)P.cap * D;
  const float* pt = P.ptab + ((long long)lane_local * R + row) * P.cap;
  const int32_t* rs = P.rec_slot + (long long)lane_local * P.block_tokens * 2;
  const float* rr = P.rec_rows + (long long)lane_local * P.block_tokens * 2 * D;
  // A record made at step k (k >= tok) holds the row of its slot as token tok attended it, unless an earlier record
  // (tok <= k' < k) of the same slot does: the first record of a slot at or after the token's own step counts.  One
  // thread per record decides that and fetches the token's probability of the slot; the channel threads then go over
  // the records without a load that depends on another.
  constexpr int kMaxRec = 16;                            // 2 * block_tokens, block_tokens <= 8
  __shared__ int rec_slot_s[kMaxRec];
  __shared__ float rec_p_s[kMaxRec];
  const int n_rec = 2 * n_act;
  if (c < kMaxRec) {
    int slot = -1;
    if (c >= 2 * tok && c < n_rec) {
      slot = rs[c];
      for (int k2 = 2 * tok; k2 < c; ++k2)
        if (rs[k2] == slot) slot = -1;
    }
    rec_slot_s[c] = slot;
    rec_p_s[c] = slot >= 0 ? pt[slot] : 0.f;
  }
  float o = 0.f;
  for (int u = 0; u < P.n_units; ++u) o += P.opart[(((long long)lane_local * P.n_units + u) * R + row) * D + c];
  __syncthreads();
#pragma unroll 4
  for (int k = 2 * tok; k < n_rec; ++k) {
    const int slot = rec_slot_s[k];                      // the same for every thread of the CTA
    if (slot >= 0) o += rec_p_s[k] * (rr[(long long)k * D + c] - to_f32(Vl[(long long)slot * D + c]));
  }
  T* dst = reinterpret_cast<T*>(P.out) + b * P.out_bs + (long long)(P.tok0 + tok) * P.out_ts + ((long long)hk * P.group + g) * D;
  dst[c] = from_f32<T>(o);
}

}  // namespace wkv
