// Host side of the C ABI declared in include/wkv.h: configuration checks, device state, launches,
// export / import of lanes.  All arithmetic of the method lives in wkv_kernels.cuh.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include <cuda.h>                      // tensor-map types only; the driver entry point is looked up at run time

#include "../../include/wkv.h"
#include "wkv_kernels.cuh"
#include "wkv_prefill.cuh"
#include "wkv_block.cuh"

struct wkv_ctx {
  wkv_config cfg;
  int device = 0;
  int lanes_per_layer = 0;
  long long lanes_total = 0;
  int cap = 0;            // slots per lane
  int group = 1;
  int n_splits = 1;       // units per lane; with the flat deal the most pieces a lane can have (stride of the partials)
  int flat_chunk = 0;     // tiles per CTA under the flat deal of the two-kernel schedule, 0 = even deal
  int chunk_cap = 0;      // cluster kernel: logits per CTA and query head
  bool use_cluster = false;
  // all layers of a step in one launch (wkv_decode_step_layers), when the scratch for every lane at once is small
  bool fused_ok = false, fused_cluster = false;
  int fused_splits = 1, fused_chunk_cap = 0, fused_flat_chunk = 0;
  float* fused_logits = nullptr;
  float* fused_part = nullptr;
  int sm_count = 148;
  float scale = 0.f;
  size_t elem = 2;
  cudaStream_t stream = nullptr;
  // device memory (provider-owned)
  void* Kc = nullptr;
  void* Vc = nullptr;
  float* a = nullptr;
  int32_t* pos = nullptr;
  int32_t* next = nullptr;
  int32_t* prev = nullptr;
  int32_t* lane_state = nullptr;
  float* logits[2] = {nullptr, nullptr};   // two scratch sets: consecutive layer calls may overlap (see prepare_overlap)
  float* part[2] = {nullptr, nullptr};
  uint32_t* ticket[2] = {nullptr, nullptr};
  uint32_t* fused_ticket = nullptr;
  int32_t* fused_seq_lens = nullptr;   // [n_layers * batch]: a caller's per-sequence lengths repeated for every layer
  int parity = 0;
  // what the previous layer call of this context wrote for the caller, and for which layer
  int last_layer = -1;
  const char* last_out[3] = {nullptr, nullptr, nullptr};
  size_t last_out_bytes[3] = {0, 0, 0};
  uint32_t* status = nullptr;
  // four query heads on bf16 rows: the scan takes its V tiles through this tensor map (see StepParams::vmap)
  alignas(64) unsigned char vmap[128] = {};
  // bf16 rows: the K and the V cache once more, in boxes of 64 rows (the dense prompt kernel's tile)
  alignas(64) unsigned char dense_kmap[128] = {};
  alignas(64) unsigned char dense_vmap[128] = {};
  // staging for the host-buffer entry point and for discarded prefill outputs
  void* stage_q = nullptr;
  void* stage_k = nullptr;
  void* stage_v = nullptr;
  void* stage_out = nullptr;
  int32_t* stage_ev = nullptr;
  // bulk prompt phase: scratch for the logits of one block of query rows per lane (taken on first use), and which
  // layers have consumed no token since creation / the last reset
  float* bulk_S = nullptr;
  int bulk_stride = 0;
  long long bulk_lanes = 0;     // lanes the scratch has rows for
  int bulk_rows = 0;            // ... logit rows per lane (16, or 32 where a launch ran blocks of 32 rows)
  // per layer: an upper bound on the tokens any lane of the layer has consumed since creation / reset; while it is
  // below the budget no lane has compressed and token i of every lane sits in slot i (kCompressed: unknown / beyond)
  // blocked prompt tail (wkv_block.cuh): scratch for `blk_lanes` lanes, taken on first use
  float* blk_logits = nullptr;
  float* blk_lgx = nullptr;
  float* blk_ptab = nullptr;
  float* blk_opart = nullptr;
  float* blk_rec_rows = nullptr;
  int32_t* blk_rec_slot = nullptr;
  long long blk_lanes = 0;
  int blk_units = 1;
  std::vector<long long> tokens_hi;
  std::vector<void*> owned;
  long long device_bytes = 0;
  long long launches = 0;
  std::string last_error;
};

// Scratch of wkv_decode_step_static.  It lives in the library image: every GPU that loads the library holds
// these bytes until the process exits.  Host code must not pass this name to a kernel -- on the host it is
// only a stand-in for the symbol; the device address comes from cudaGetSymbolAddress (static_scratch_base).
constexpr size_t kStaticScratchBytes = (size_t)WKV_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {

int fail(wkv_ctx* c, int code, const std::string& msg) {
  if (c) c->last_error = msg;
  return code;
}
int cuda_fail(wkv_ctx* c, cudaError_t e, const char* what) {
  return fail(c, WKV_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}
#define WKV_CUDA(ctx, expr)                                   \
  do {                                                        \
    cudaError_t e_ = (expr);                                  \
    if (e_ != cudaSuccess) return cuda_fail(ctx, e_, #expr);  \
  } while (0)

void* default_alloc(size_t bytes, void*) {
  void* p = nullptr;
  if (cudaMalloc(&p, bytes) != cudaSuccess) return nullptr;
  return p;
}
void default_release(void* p, void*) { cudaFree(p); }

template <typename P>
int take(wkv_ctx* c, P** dst, size_t bytes) {
  bytes = (bytes + 255) & ~(size_t)255;
  void* p = c->cfg.alloc(bytes, c->cfg.user);
  if (!p) return fail(c, WKV_ERR_ALLOC, "device memory provider returned NULL for " + std::to_string(bytes) + " bytes");
  c->owned.push_back(p);
  c->device_bytes += (long long)bytes;
  *dst = reinterpret_cast<P*>(p);
  return WKV_OK;
}

// Tensor maps.  The driver's encoder is found through the runtime: the library does not link against the driver.
// encode_value_map: the value cache as a [rows][head_dim] bf16 matrix, boxes of 64 elements x one scan tile of rows.
int encode_rows_map(wkv_ctx* c, unsigned char* out128, const void* base, unsigned long long row_elems, unsigned long long rows,
                    unsigned box_rows);
int encode_value_map(wkv_ctx* c, void* base, unsigned long long rows, int head_dim) {
  if (rows >= 0x7fffffffULL) return fail(c, WKV_ERR_INVALID, "n_layers * batch * n_kv_heads * (budget + 1) must stay below 2^31 rows with bf16 storage");
  return encode_rows_map(c, c->vmap, base, (unsigned long long)head_dim, rows, (unsigned)wkv::kTileSlots);
}
// bf16 matrix [rows][row_elems] (row-major, rows 16-byte aligned), boxes of 64 elements x box_rows rows, 128-byte swizzle,
// zero fill outside the matrix.
int encode_rows_map(wkv_ctx* c, unsigned char* out128, const void* base, unsigned long long row_elems, unsigned long long rows,
                    unsigned box_rows) {
  typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static_assert(sizeof(CUtensorMap) == sizeof(c->vmap), "tensor map size");
  void* sym = nullptr;
  cudaDriverEntryPointQueryResult qr = cudaDriverEntryPointSymbolNotFound;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qr);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)");
  if (qr != cudaDriverEntryPointSuccess || !sym) return fail(c, WKV_ERR_CUDA, "the driver has no cuTensorMapEncodeTiled");
  const cuuint64_t dims[2] = {(cuuint64_t)row_elems, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)row_elems * 2};
  const cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1u, 1u};
  CUtensorMap m;
  const CUresult r = reinterpret_cast<encode_fn>(sym)(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                                                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(c, WKV_ERR_CUDA, "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r));
  std::memcpy(out128, &m, sizeof(m));
  return WKV_OK;
}

const char* check_config(const wkv_config* c) {
  if (!c) return "config is NULL";
  if (c->n_layers < 1 || c->batch < 1) return "n_layers and batch must be >= 1";
  if (c->n_kv_heads < 1 || c->n_q_heads < 1 || c->n_q_heads % c->n_kv_heads) return "n_q_heads must be a positive multiple of n_kv_heads";
  const int g = c->n_q_heads / c->n_kv_heads;
  if (g != 1 && g != 2 && g != 4 && g != 8) return "n_q_heads / n_kv_heads must be 1, 2, 4 or 8";
  if (c->head_dim != 64 && c->head_dim != 128) return "head_dim must be 64 or 128";
  if (c->dtype != WKV_F32 && c->dtype != WKV_BF16) return "dtype must be WKV_F32 or WKV_BF16";
  if (c->budget < 1 || c->budget >= (1 << 20)) return "budget must be in [1, 2^20)";
  if (c->window < 1) return "window must be >= 1 (the newest entry has no right neighbour)";
  if (c->sink < 0) return "sink must be >= 0";
  if ((long long)c->sink + c->window > c->budget) return "budget must be >= sink + window";
  if (c->merge != 0 && c->merge != 1) return "merge must be 0 or 1";
  if (c->n_splits < 0 || c->n_splits > wkv::kMaxSplits) return "n_splits must be in [0, 64]";
  if (!(c->scale >= 0.f) || std::isinf(c->scale)) return "scale must be finite and >= 0";
  if (c->schedule < WKV_SCHEDULE_AUTO || c->schedule > WKV_SCHEDULE_FLAT) return "schedule must be 0 (auto), 1 (two kernels), 2 (clusters) or 3 (two kernels, flat deal)";
  if ((c->alloc == nullptr) != (c->release == nullptr)) return "alloc and release must both be set or both be NULL";
  if ((long long)c->batch * c->n_kv_heads * wkv::kMaxSplits > 0x7fffffffLL) return "batch * n_kv_heads too large";
  return nullptr;
}

// Scan CTAs that fit on one SM together (registers and shared memory of the instantiation this configuration runs;
// flat: the entry of the flat deal).
template <typename T, int D, int G>
int scan_ctas_per_sm_of(bool flat) {
  int n = 0;
  constexpr int smem = wkv::scan_smem_bytes<T, D, G>();
  if (cudaFuncSetAttribute(wkv::scan_entry<T, D, G>(flat), cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, wkv::scan_entry<T, D, G>(flat), wkv::kThreads, smem) != cudaSuccess) {
    cudaGetLastError();
    return 4;
  }
  return n < 1 ? 1 : n;
}
template <typename T, int D>
int scan_ctas_per_sm_by_group(int G, bool flat) {
  switch (G) {
    case 1: return scan_ctas_per_sm_of<T, D, 1>(flat);
    case 2: return scan_ctas_per_sm_of<T, D, 2>(flat);
    case 4: return scan_ctas_per_sm_of<T, D, 4>(flat);
    default: return scan_ctas_per_sm_of<T, D, 8>(flat);
  }
}
int scan_ctas_per_sm(const wkv_config& c, bool flat) {
  const int G = c.n_q_heads / c.n_kv_heads;
  if (c.dtype == WKV_BF16) return c.head_dim == 128 ? scan_ctas_per_sm_by_group<__nv_bfloat16, 128>(G, flat) : scan_ctas_per_sm_by_group<__nv_bfloat16, 64>(G, flat);
  return c.head_dim == 128 ? scan_ctas_per_sm_by_group<float, 128>(G, flat) : scan_ctas_per_sm_by_group<float, 64>(G, flat);
}

// Splits per lane when the caller leaves the choice to the library: a power of two (so the lane's CTAs can form a
// thread-block cluster), enough CTAs to fill 148 SMs several times over, at least ~4 tiles of work per CTA.
// `slots` = scan CTAs the whole GPU holds at once.
int auto_splits(const wkv_config& c, long long lanes, long long slots) {
  const int tiles = (c.budget + 1 + wkv::kTileSlots - 1) / wkv::kTileSlots;
  int s = 1;
  while (s < 16 && lanes * s < 1776 && tiles / (2 * s) >= 4) s *= 2;
  if (c.schedule != WKV_SCHEDULE_CLUSTER && lanes * tiles >= 148 * 64) {
    // two-kernel schedule: units of about 32 tiles balance the SMs and amortise each CTA's start-up
    s = (tiles + 31) / 32;
    if (s > wkv::kMaxSplits) s = wkv::kMaxSplits;
    if (s < 1) s = 1;
    // ... unless the units then fill the last round of resident CTAs badly: a layer's time is about (rounds of resident
    // CTAs) x (tiles per unit + a start-up of ~3 tiles); take the split count that makes that product clearly smaller.
    auto cost = [&](int k) { return ((lanes * k + slots - 1) / slots) * ((tiles + k - 1) / k + 3); };
    int best = s;
    for (int k = 1; k <= 16 && tiles / k >= 8; ++k)
      if (cost(k) < cost(best)) best = k;
    if (cost(best) * 26 < cost(s) * 25) s = best;
  }
  return s;
}

bool is_cluster_size(int s) { return s == 1 || s == 2 || s == 4 || s == 8 || s == 16; }

// The flat deal of the two-kernel schedule (see lane_pieces in wkv_kernels.cuh): tiles per CTA, or 0 to keep whole units
// per lane.  `units` = the even deal's split count.  Chosen when the even deal would put all its CTAs on the GPU in one
// wave that fills the SMs unequally -- then the slowest SM sets the time -- or when the caller asks for it; on request
// n_splits > 0 means that many CTAs per lane on average.  slots / flat_slots: scan CTAs the GPU holds at once under either
// deal.  `stride` receives the most pieces a lane can have.
int flat_deal(const wkv_config& c, long long lanes, long long slots, long long flat_slots, int sms, int units, int* stride) {
  const int tiles = (c.budget + 1 + wkv::kTileSlots - 1) / wkv::kTileSlots;
  const long long total = lanes * tiles;
  long long n_ctas;
  if (c.schedule == WKV_SCHEDULE_FLAT) {
    n_ctas = c.n_splits > 0 ? lanes * c.n_splits : flat_slots;
  } else {
    if (c.schedule != WKV_SCHEDULE_AUTO || c.n_splits > 0) return 0;
    // Only where the scan is bound by instruction issue, i.e. per SM: four or more query heads per cache row.  A
    // bandwidth-bound scan shares HBM among all SMs, so an SM holding fewer CTAs simply finishes each of them sooner,
    // and whole units keep the start-up cost lower (measured: one head per row, 256 lanes x 52 tiles, 44.3 us per layer
    // call with whole units against 45.2 us flat; four heads per row, 256 lanes x 103 tiles, 99.2 against 96.6 us).
    if (c.n_q_heads / c.n_kv_heads < 4) return 0;
    const long long even = lanes * units;
    if (even > slots || even <= sms || even % sms == 0) return 0;        // several waves, or already level
    // whole CTAs per SM, at least 8 tiles each
    const long long per_sm = std::min<long long>(flat_slots / sms, total / (8LL * sms));
    if (per_sm < 1) return 0;
    n_ctas = per_sm * sms;
  }
  if (n_ctas < 1) n_ctas = 1;
  long long chunk = (total + n_ctas - 1) / n_ctas;
  chunk = std::max<long long>(chunk, (tiles + wkv::kMaxSplits - 3) / (wkv::kMaxSplits - 2));   // at most kMaxSplits pieces per lane
  if (chunk < 1) chunk = 1;
  if (chunk > 0x3fffffff) return 0;
  *stride = (int)((tiles + chunk - 1) / chunk) + 1;
  if (*stride > wkv::kMaxSplits) return 0;
  return (int)chunk;
}

constexpr int kMaxDynSmem = 200 * 1024;

// Threads per lane of the lane-epilogue kernel for a launch of `lanes` lanes: 512 (one or two query heads) or 384 (four)
// when two such CTAs per SM hold every lane at once, else 256.
inline int epilogue_threads(int G, int lanes, int sms) {
  if (G <= 2 && lanes <= 2 * sms) return wkv::kEpilogueThreadsWide;
  if (G == 4 && lanes <= 2 * sms) return wkv::kEpilogueThreadsMid;
  return wkv::kEpilogueThreads;
}

// The lane-epilogue kernel: one CTA per lane, launched with programmatic stream serialization (it orders itself
// against its predecessor on the device).
template <typename T, int D, int G>
cudaError_t launch_epilogue(const wkv::StepParams& P, int lanes, int dev, cudaStream_t stream, bool whole_block = false) {
  cudaLaunchAttribute pdl[1];
  pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  pdl[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t k2 = {};
  k2.gridDim = dim3((unsigned)lanes);
  int sms = 148;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int nt = epilogue_threads(G, lanes, sms);
  k2.blockDim = dim3(nt);
  k2.stream = stream;
  k2.attrs = pdl;
  k2.numAttrs = 1;
  // room to stage a lane's scores and positions in shared memory, when the lane can be finished out of registers
  wkv::StepParams P2 = P;
  const int e_slots = wkv::epilogue_slots_per_thread(G, nt) * nt;
  P2.ep_stage_slots = (e_slots > 0 && P.budget + 1 <= e_slots) ? P.cap : 0;
  k2.dynamicSmemBytes = (size_t)P2.ep_stage_slots * 8;
  if (whole_block) {
    // every token of a block of a blocked prompt tail in one launch (lane_epilogue_block_kernel)
    if constexpr (G <= 2) {
      if (nt == wkv::kEpilogueThreadsWide) return cudaLaunchKernelEx(&k2, wkv::lane_epilogue_block_kernel<T, D, G, wkv::kEpilogueThreadsWide>, P2);
    }
    if constexpr (G == 4) {
      if (nt == wkv::kEpilogueThreadsMid) return cudaLaunchKernelEx(&k2, wkv::lane_epilogue_block_kernel_mid<T, D, G>, P2);
    }
    if constexpr (G <= 4) return cudaLaunchKernelEx(&k2, wkv::lane_epilogue_block_kernel<T, D, G, wkv::kEpilogueThreads>, P2);
    return cudaErrorInvalidValue;
  }
  if constexpr (G <= 2) {
    if (nt == wkv::kEpilogueThreadsWide) return cudaLaunchKernelEx(&k2, wkv::lane_epilogue_kernel<T, D, G, wkv::kEpilogueThreadsWide>, P2);
  }
  if constexpr (G == 4) {
    if (nt == wkv::kEpilogueThreadsMid) return cudaLaunchKernelEx(&k2, wkv::lane_epilogue_kernel_mid<T, D, G>, P2);
  }
  return cudaLaunchKernelEx(&k2, wkv::lane_epilogue_kernel<T, D, G, wkv::kEpilogueThreads>, P2);
}

// cluster = true: one launch, the n_splits CTAs of a lane form a thread-block cluster;
// otherwise two launches: the scan over all units, then one CTA per lane on the finished scratch.
template <typename T, int D, int G>
cudaError_t launch_step(const wkv::StepParams& P, int lanes, bool cluster, cudaStream_t stream) {
  using C = wkv::Cfg<T, D, G>;
  // largest dynamic shared memory size configured per device and kernel (contexts may be driven from several host
  // threads: two of them setting the same attribute twice is harmless, a torn read is not)
  static std::atomic<int> attr_done[64][3];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  const int smem = cluster ? C::kFixedBytes + G * P.chunk_cap * 4 : wkv::scan_smem_bytes<T, D, G>();
  if (smem > kMaxDynSmem) return cudaErrorInvalidValue;
  const bool flat = !cluster && P.flat_chunk > 0;
  const int which = cluster ? 1 : (flat ? 2 : 0);
  const void* fn = cluster ? (const void*)wkv::decode_step_cluster_kernel<T, D, G> : (const void*)wkv::scan_entry<T, D, G>(flat);
  if (attr_done[dev][which].load(std::memory_order_acquire) < smem) {
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    if (cluster) {
      e = cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      if (e != cudaSuccess) return e;
    }
    attr_done[dev][which].store(smem, std::memory_order_release);
  }
  const int n_ctas = P.flat_chunk > 0 ? (int)(((long long)lanes * P.tiles_cap + P.flat_chunk - 1) / P.flat_chunk) : lanes * P.n_splits;
  if (!cluster) {
    // Both kernels are launched with programmatic stream serialization: each may be set up while its predecessor
    // drains and orders itself against it on the device (griddep_wait in the kernels).
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t k1 = {};
    k1.gridDim = dim3((unsigned)n_ctas);
    k1.blockDim = dim3(wkv::kThreads);
    k1.dynamicSmemBytes = (size_t)smem;
    k1.stream = stream;
    k1.attrs = pdl;
    k1.numAttrs = 1;
    e = cudaLaunchKernelEx(&k1, wkv::scan_entry<T, D, G>(flat), P);
    if (e != cudaSuccess) return e;
    return launch_epilogue<T, D, G>(P, lanes, dev, stream);
  }
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3((unsigned)n_ctas);
  lc.blockDim = dim3(wkv::kThreads);
  lc.dynamicSmemBytes = (size_t)smem;
  lc.stream = stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)P.n_splits;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // the kernel waits for its predecessor first thing
  at[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = 2;
  return cudaLaunchKernelEx(&lc, wkv::decode_step_cluster_kernel<T, D, G>, P);
}

template <typename T, int D>
cudaError_t launch_by_group(int G, const wkv::StepParams& P, int lanes, bool cluster, cudaStream_t s) {
  switch (G) {
    case 1: return launch_step<T, D, 1>(P, lanes, cluster, s);
    case 2: return launch_step<T, D, 2>(P, lanes, cluster, s);
    case 4: return launch_step<T, D, 4>(P, lanes, cluster, s);
    case 8: return launch_step<T, D, 8>(P, lanes, cluster, s);
  }
  return cudaErrorInvalidValue;
}

// cluster = false forces the two-kernel schedule (global scratch), which the static-scratch entry point needs.
cudaError_t launch_any(const wkv_ctx* c, const wkv::StepParams& P_in, bool cluster, int lanes = 0) {
  const int n = lanes > 0 ? lanes : c->lanes_per_layer;
  wkv::StepParams P = P_in;
  P.n_lanes = n;
  if (cluster) P.flat_chunk = 0;
  if (c->cfg.dtype == WKV_BF16) {
    return c->cfg.head_dim == 128 ? launch_by_group<__nv_bfloat16, 128>(c->group, P, n, cluster, c->stream)
                                  : launch_by_group<__nv_bfloat16, 64>(c->group, P, n, cluster, c->stream);
  }
  return c->cfg.head_dim == 128 ? launch_by_group<float, 128>(c->group, P, n, cluster, c->stream)
                                : launch_by_group<float, 64>(c->group, P, n, cluster, c->stream);
}

wkv::StepParams base_params(const wkv_ctx* c, int layer) {
  wkv::StepParams P;
  std::memset(&P, 0, sizeof(P));
  P.Kc = c->Kc; P.Vc = c->Vc; P.a = c->a; P.pos = c->pos; P.next = c->next; P.prev = c->prev;
  P.lane_state = c->lane_state; P.logits = c->logits[0]; P.part = c->part[0]; P.status = c->status;
  P.lane0 = layer * c->lanes_per_layer;
  P.n_kv_heads = c->cfg.n_kv_heads;
  P.cap = c->cap;
  P.budget = c->cfg.budget; P.window = c->cfg.window; P.sink = c->cfg.sink;
  P.n_splits = c->n_splits;
  P.flat_chunk = c->flat_chunk;
  P.tiles_cap = (c->cfg.budget + 1 + wkv::kTileSlots - 1) / wkv::kTileSlots;
  P.chunk_cap = c->chunk_cap;
  P.merge = c->cfg.merge;
  P.scale = c->scale;
  P.logit_rows = c->group;
  P.probs_rows = c->group;
  P.probs_stride = c->cfg.budget + 1;
  std::memcpy(P.vmap, c->vmap, sizeof(P.vmap));
  return P;
}

bool ranges_overlap(const void* a, size_t na, const void* b, size_t nb) {
  if (!a || !b || !na || !nb) return false;
  const char* x = (const char*)a;
  const char* y = (const char*)b;
  return x < y + nb && y < x + na;
}

// The context whose kernels were the last ones this library launched (see prepare_overlap).
std::atomic<const wkv_ctx*> g_last_launcher{nullptr};

// Two-kernel schedule: choose the scratch set of this layer call and decide whether its scan may start while the
// previous call's lane epilogue is still running.  Only a caller that vouches for its inputs (inputs_ready: q, k, v of
// this call were complete before the previous layer call was issued -- wkv_decode_step_layers) can get that overlap,
// and then only if the previous call of this context was for another layer, no other context launched in between,
// and this call's inputs do not alias what the previous call wrote for the caller.  A scan behind a foreign kernel
// always waits for it first: nothing is known about when that kernel's results become visible.
void prepare_overlap(wkv_ctx* c, wkv::StepParams& P, int layer, size_t q_bytes, size_t kv_bytes, bool inputs_ready) {
  c->parity ^= 1;
  P.logits = c->logits[c->parity];
  P.part = c->part[c->parity];
  P.ticket = c->ticket[c->parity];
  // 2: the previous kernel may touch this layer's lanes or is unknown; 1: it cannot, but it may be what produces this
  // call's inputs; 0: the caller vouches for the inputs and they do not alias the previous call's outputs.
  int level = (c->last_layer < 0 || c->last_layer == layer || g_last_launcher.load() != c) ? 2 : (inputs_ready ? 0 : 1);
  for (int i = 0; i < 3 && level == 0; ++i) {
    if (ranges_overlap(P.q, q_bytes, c->last_out[i], c->last_out_bytes[i]) ||
        ranges_overlap(P.k, kv_bytes, c->last_out[i], c->last_out_bytes[i]) ||
        ranges_overlap(P.v, kv_bytes, c->last_out[i], c->last_out_bytes[i]))
      level = 1;
  }
  P.wait_at_start = level;
  c->last_layer = layer;
  g_last_launcher.store(c);
}

void note_outputs(wkv_ctx* c, const void* out, size_t out_bytes, const void* ev, size_t ev_bytes, const void* probs,
                  size_t probs_bytes) {
  c->last_out[0] = (const char*)out;   c->last_out_bytes[0] = out_bytes;
  c->last_out[1] = (const char*)ev;    c->last_out_bytes[1] = ev_bytes;
  c->last_out[2] = (const char*)probs; c->last_out_bytes[2] = probs_bytes;
}

int run_reset(wkv_ctx* c) {
  c->tokens_hi.assign((size_t)c->cfg.n_layers, 0);
  for (int i = 0; i < 2; ++i) WKV_CUDA(c, cudaMemsetAsync(c->ticket[i], 0, (size_t)c->lanes_per_layer * 4, c->stream));
  if (c->fused_ticket) WKV_CUDA(c, cudaMemsetAsync(c->fused_ticket, 0, (size_t)c->lanes_total * 4, c->stream));
  wkv::reset_kernel<<<592, 256, 0, c->stream>>>(c->lane_state, c->pos, c->a, c->next, c->prev, c->lanes_total, c->cap,
                                                c->status);
  c->launches++;
  WKV_CUDA(c, cudaGetLastError());
  return WKV_OK;
}

// Device address of g_static_scratch on the current device, looked up once per device.
cudaError_t static_scratch_base(unsigned char** base) {
  static std::atomic<unsigned char*> per_device[64];       // zero-initialised; every thread would store the same address
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  unsigned char* p = per_device[dev].load(std::memory_order_acquire);
  if (p == nullptr) {
    e = cudaGetSymbolAddress((void**)&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    per_device[dev].store(p, std::memory_order_release);
  }
  *base = p;
  return cudaSuccess;
}

int check_lane(wkv_ctx* c, int layer, int b, int h) {
  if (!c) return WKV_ERR_INVALID;
  if (layer < 0 || layer >= c->cfg.n_layers || b < 0 || b >= c->cfg.batch || h < 0 || h >= c->cfg.n_kv_heads)
    return fail(c, WKV_ERR_INVALID, "layer / sequence / kv_head out of range");
  return WKV_OK;
}

template <typename T, int D, int KT, int ROWS = wkv::kBulkRows>
cudaError_t launch_bulk(int G, const wkv::PrefillParams& P, int lanes, cudaStream_t s) {
  constexpr int smem = wkv::bulk_smem_bytes<T, D, KT, ROWS>();
  auto go = [&](auto kern) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    kern<<<lanes, wkv::bulk_threads(ROWS), smem, s>>>(P);
    return cudaGetLastError();
  };
  switch (G) {
    case 1: return go(wkv::prefill_bulk_kernel<T, D, 1, KT, ROWS>);
    case 2: return go(wkv::prefill_bulk_kernel<T, D, 2, KT, ROWS>);
    case 4: return go(wkv::prefill_bulk_kernel<T, D, 4, KT, ROWS>);
    case 8: return go(wkv::prefill_bulk_kernel<T, D, 8, KT, ROWS>);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

extern "C" {

const char* wkv_config_error(const wkv_config* cfg) { return check_config(cfg); }

int wkv_create(const wkv_config* cfg, wkv_ctx** out) {
  if (!out) return WKV_ERR_INVALID;
  *out = nullptr;
  if (check_config(cfg) != nullptr) return WKV_ERR_INVALID;
  wkv_ctx* c = new (std::nothrow) wkv_ctx;
  if (!c) return WKV_ERR_ALLOC;
  c->cfg = *cfg;
  if (!c->cfg.alloc) { c->cfg.alloc = default_alloc; c->cfg.release = default_release; c->cfg.user = nullptr; }
  cudaError_t e = cudaGetDevice(&c->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
  if (e != cudaSuccess) { delete c; return WKV_ERR_CUDA; }
  c->group = cfg->n_q_heads / cfg->n_kv_heads;
  c->lanes_per_layer = cfg->batch * cfg->n_kv_heads;
  c->lanes_total = (long long)cfg->n_layers * c->lanes_per_layer;
  c->cap = (cfg->budget + 1 + 3) & ~3;
  const long long slots = (long long)c->sm_count * scan_ctas_per_sm(*cfg, false);
  const long long flat_slots = (long long)c->sm_count * scan_ctas_per_sm(*cfg, true);
  c->n_splits = cfg->n_splits > 0 ? cfg->n_splits : auto_splits(*cfg, c->lanes_per_layer, slots);
  {
    const int tiles = (cfg->budget + 1 + wkv::kTileSlots - 1) / wkv::kTileSlots;
    c->chunk_cap = ((tiles + c->n_splits - 1) / c->n_splits) * wkv::kTileSlots;   // the largest share of an even deal
    // kernel B needs a cluster-sized split count and room for the chunk's logits next to the ring
    const bool can_cluster = is_cluster_size(c->n_splits) && c->group * c->chunk_cap * 4 <= 64 * 1024;
    if (cfg->schedule == WKV_SCHEDULE_CLUSTER && !can_cluster) {
      delete c;
      return WKV_ERR_INVALID;
    }
    // a handful of lanes: latency is everything, one launch and a cluster sharing the lane's epilogue (measured:
    // 10.8 vs 14.2 us per step on 4 lanes x 5 tiles); otherwise scan all units with short-lived CTAs and finish the
    // lanes in a second launch (17.4 vs 18.4 us on 32 lanes x 65 tiles, and far ahead on large shapes)
    c->use_cluster = cfg->schedule == WKV_SCHEDULE_CLUSTER ||
                     (cfg->schedule == WKV_SCHEDULE_AUTO && can_cluster && c->lanes_per_layer * tiles < 148 * 4);
    if (!c->use_cluster) {
      int stride = 0;
      const int chunk = flat_deal(*cfg, c->lanes_per_layer, slots, flat_slots, c->sm_count, c->n_splits, &stride);
      if (chunk > 0) { c->flat_chunk = chunk; c->n_splits = stride; }
    }
  }
  if (cfg->n_layers > 1 && c->lanes_total * wkv::kMaxSplits < 0x7fffffffLL) {
    // One launch for all layers: the lanes of all layers are just more lanes.  Worth it when a layer alone cannot
    // fill the GPU; allowed when the scratch for every lane at once stays small.
    const int tiles = (cfg->budget + 1 + wkv::kTileSlots - 1) / wkv::kTileSlots;
    c->fused_splits = cfg->n_splits > 0 ? cfg->n_splits : auto_splits(*cfg, c->lanes_total, slots);
    c->fused_chunk_cap = ((tiles + c->fused_splits - 1) / c->fused_splits) * wkv::kTileSlots;
    const bool can_cluster = is_cluster_size(c->fused_splits) && c->group * c->fused_chunk_cap * 4 <= 64 * 1024;
    c->fused_cluster = cfg->schedule == WKV_SCHEDULE_CLUSTER ? can_cluster
                       : (cfg->schedule == WKV_SCHEDULE_AUTO && can_cluster && c->lanes_total * tiles < 148 * 4);
    if (!c->fused_cluster) {
      int stride = 0;
      const int chunk = flat_deal(*cfg, c->lanes_total, slots, flat_slots, c->sm_count, c->fused_splits, &stride);
      if (chunk > 0) { c->fused_flat_chunk = chunk; c->fused_splits = stride; }
    }
    const size_t bytes = (size_t)c->lanes_total * c->group * ((size_t)c->cap * 4 + (size_t)c->fused_splits * (cfg->head_dim + 2) * 4);
    c->fused_ok = bytes <= ((size_t)64 << 20) && (cfg->schedule != WKV_SCHEDULE_CLUSTER || can_cluster);
  }
  c->scale = cfg->scale != 0.f ? cfg->scale : (float)(1.0 / std::sqrt((double)cfg->head_dim));
  c->elem = cfg->dtype == WKV_BF16 ? 2 : 4;
  c->stream = reinterpret_cast<cudaStream_t>(cfg->stream);

  const size_t D = cfg->head_dim, cap = c->cap, G = c->group;
  const size_t row = D * c->elem;
  int rc = WKV_OK;
  // one request after the other; after the first refusal the provider is not asked again
#define WKV_TAKE(dst, bytes) do { if (rc == WKV_OK) rc = take(c, dst, bytes); } while (0)
  WKV_TAKE(&c->Kc, (size_t)c->lanes_total * cap * row);
  WKV_TAKE(&c->Vc, (size_t)c->lanes_total * cap * row);
  WKV_TAKE(&c->a, (size_t)c->lanes_total * cap * 4);
  WKV_TAKE(&c->pos, (size_t)c->lanes_total * cap * 4);
  WKV_TAKE(&c->next, (size_t)c->lanes_total * cap * 4);
  WKV_TAKE(&c->prev, (size_t)c->lanes_total * cap * 4);
  WKV_TAKE(&c->lane_state, (size_t)c->lanes_total * wkv::LS_STRIDE * 4);
  for (int i = 0; i < 2; ++i) {
    WKV_TAKE(&c->logits[i], (size_t)c->lanes_per_layer * G * cap * 4);
    WKV_TAKE(&c->part[i], (size_t)c->lanes_per_layer * c->n_splits * G * (D + 2) * 4);
    WKV_TAKE(&c->ticket[i], (size_t)c->lanes_per_layer * 4);
  }
  if (c->fused_ok) {
    WKV_TAKE(&c->fused_logits, (size_t)c->lanes_total * G * cap * 4);
    WKV_TAKE(&c->fused_part, (size_t)c->lanes_total * c->fused_splits * G * (D + 2) * 4);
    WKV_TAKE(&c->fused_ticket, (size_t)c->lanes_total * 4);
    WKV_TAKE(&c->fused_seq_lens, (size_t)cfg->n_layers * cfg->batch * 4);
  }
  WKV_TAKE(&c->status, 256);
  // staging holds one step of all layers (the host entry points copy through it)
  WKV_TAKE(&c->stage_q, (size_t)cfg->n_layers * cfg->batch * cfg->n_q_heads * row);
  WKV_TAKE(&c->stage_k, (size_t)c->lanes_total * row);
  WKV_TAKE(&c->stage_v, (size_t)c->lanes_total * row);
  WKV_TAKE(&c->stage_out, (size_t)cfg->n_layers * cfg->batch * cfg->n_q_heads * row);
  WKV_TAKE(&c->stage_ev, (size_t)c->lanes_total * 4);
#undef WKV_TAKE
  // bf16 rows: the scan with four query heads per key and the value sweep of a blocked prompt tail take V tiles through it
  if (rc == WKV_OK && cfg->dtype == WKV_BF16)
    rc = encode_value_map(c, c->Vc, (unsigned long long)c->lanes_total * cap, cfg->head_dim);
  if (rc == WKV_OK && cfg->dtype == WKV_BF16)
    rc = encode_rows_map(c, c->dense_kmap, c->Kc, (unsigned long long)cfg->head_dim, (unsigned long long)c->lanes_total * cap, 64u);
  if (rc == WKV_OK && cfg->dtype == WKV_BF16)
    rc = encode_rows_map(c, c->dense_vmap, c->Vc, (unsigned long long)cfg->head_dim, (unsigned long long)c->lanes_total * cap, 64u);
  if (rc == WKV_OK) rc = run_reset(c);
  if (rc != WKV_OK) {
    wkv_destroy(c);
    return rc;
  }
  *out = c;
  return WKV_OK;
}

void wkv_destroy(wkv_ctx* c) {
  if (!c) return;
  cudaStreamSynchronize(c->stream);
  for (void* p : c->owned) c->cfg.release(p, c->cfg.user);
  delete c;
}

int wkv_reset(wkv_ctx* c) {
  if (!c) return WKV_ERR_INVALID;
  c->last_layer = -1;
  return run_reset(c);
}

int wkv_set_stream(wkv_ctx* c, void* stream) {
  if (!c) return WKV_ERR_INVALID;
  c->last_layer = -1;                  // nothing is known about what runs on the new stream
  c->stream = reinterpret_cast<cudaStream_t>(stream);
  return WKV_OK;
}

static int decode_step_impl(wkv_ctx* c, int32_t layer, const void* q, const void* k, const void* v, void* out,
                            int32_t* evicted_pos, float* probs, bool inputs_ready) {
  if (!c) return WKV_ERR_INVALID;
  if (!q || !k || !v || !out) return fail(c, WKV_ERR_INVALID, "q, k, v and out must not be NULL");
  if (layer < 0 || layer >= c->cfg.n_layers) return fail(c, WKV_ERR_INVALID, "layer out of range");
  wkv::StepParams P = base_params(c, layer);
  const long long D = c->cfg.head_dim;
  P.q = q; P.k = k; P.v = v; P.out = out; P.evicted = evicted_pos; P.probs = probs;
  P.q_bs = (long long)c->cfg.n_q_heads * D;
  P.kv_bs = (long long)c->cfg.n_kv_heads * D;
  P.out_bs = P.q_bs;
  P.ev_bs = c->cfg.n_kv_heads;
  P.seq_lens = nullptr;
  P.tok_idx = 0;
  const size_t row = (size_t)D * c->elem;
  const size_t q_bytes = (size_t)c->cfg.batch * c->cfg.n_q_heads * row, kv_bytes = (size_t)c->lanes_per_layer * row;
  c->tokens_hi[layer] += 1;
  if (!c->use_cluster) prepare_overlap(c, P, layer, q_bytes, kv_bytes, inputs_ready);
  cudaError_t e = launch_any(c, P, c->use_cluster);
  c->launches += c->use_cluster ? 1 : 2;
  if (e != cudaSuccess) return cuda_fail(c, e, "decode step launch");
  note_outputs(c, out, q_bytes, evicted_pos, (size_t)c->lanes_per_layer * 4, probs,
               (size_t)c->cfg.batch * c->cfg.n_q_heads * (c->cfg.budget + 1) * 4);
  return WKV_OK;
}

int wkv_decode_step(wkv_ctx* c, int32_t layer, const void* q, const void* k, const void* v, void* out,
                    int32_t* evicted_pos, float* probs) {
  return decode_step_impl(c, layer, q, k, v, out, evicted_pos, probs, false);
}

int wkv_decode_step_layers(wkv_ctx* c, const void* q, const void* k, const void* v, void* out, int32_t* evicted_pos) {
  if (!c) return WKV_ERR_INVALID;
  if (!q || !k || !v || !out) return fail(c, WKV_ERR_INVALID, "q, k, v and out must not be NULL");
  const size_t row = (size_t)c->cfg.head_dim * c->elem;
  const size_t q_bytes = (size_t)c->cfg.batch * c->cfg.n_q_heads * row, kv_bytes = (size_t)c->lanes_per_layer * row;
  const size_t nl = (size_t)c->cfg.n_layers;
  // the whole output range belongs to this call: a later layer's inputs must not alias an earlier layer's outputs
  if (ranges_overlap(q, q_bytes * nl, out, q_bytes * nl) || ranges_overlap(k, kv_bytes * nl, out, q_bytes * nl) ||
      ranges_overlap(v, kv_bytes * nl, out, q_bytes * nl) ||
      ranges_overlap(q, q_bytes * nl, evicted_pos, (size_t)c->lanes_per_layer * 4 * nl) ||
      ranges_overlap(k, kv_bytes * nl, evicted_pos, (size_t)c->lanes_per_layer * 4 * nl) ||
      ranges_overlap(v, kv_bytes * nl, evicted_pos, (size_t)c->lanes_per_layer * 4 * nl))
    return fail(c, WKV_ERR_INVALID, "wkv_decode_step_layers: inputs and outputs must not overlap");
  c->last_layer = -1;                   // the first layer's scan orders itself behind whatever ran before this call
  if (c->fused_ok) {
    // the lanes of all layers in one launch (pair): [n_layers, batch, ...] is [n_layers*batch, ...] to the kernels
    wkv::StepParams P = base_params(c, 0);
    P.n_splits = c->fused_splits;
    P.flat_chunk = c->fused_flat_chunk;
    P.chunk_cap = c->fused_chunk_cap;
    P.logits = c->fused_logits;
    P.part = c->fused_part;
    P.ticket = c->fused_ticket;
    P.q = q; P.k = k; P.v = v; P.out = out; P.evicted = evicted_pos; P.probs = nullptr;
    P.q_bs = (long long)c->cfg.n_q_heads * c->cfg.head_dim;
    P.kv_bs = (long long)c->cfg.n_kv_heads * c->cfg.head_dim;
    P.out_bs = P.q_bs;
    P.ev_bs = c->cfg.n_kv_heads;
    P.wait_at_start = 2;
    g_last_launcher.store(c);
    for (auto& th : c->tokens_hi) th += 1;
    cudaError_t e = launch_any(c, P, c->fused_cluster, (int)c->lanes_total);
    c->launches += c->fused_cluster ? 1 : 2;
    if (e != cudaSuccess) return cuda_fail(c, e, "decode step launch (all layers)");
    note_outputs(c, nullptr, 0, nullptr, 0, nullptr, 0);
    return WKV_OK;
  }
  for (int layer = 0; layer < c->cfg.n_layers; ++layer) {
    int rc = decode_step_impl(c, layer, (const char*)q + layer * q_bytes, (const char*)k + layer * kv_bytes,
                              (const char*)v + layer * kv_bytes, (char*)out + layer * q_bytes,
                              evicted_pos ? evicted_pos + (size_t)layer * c->lanes_per_layer : nullptr, nullptr, true);
    if (rc != WKV_OK) return rc;
  }
  c->last_layer = -1;
  return WKV_OK;
}

int wkv_decode_step_static(wkv_ctx* c, int32_t layer, const void* q, const void* k, const void* v, void* out,
                           int32_t* evicted_pos) {
  if (!c) return WKV_ERR_INVALID;
  if (!q || !k || !v || !out) return fail(c, WKV_ERR_INVALID, "q, k, v and out must not be NULL");
  if (layer < 0 || layer >= c->cfg.n_layers) return fail(c, WKV_ERR_INVALID, "layer out of range");
  const size_t D = c->cfg.head_dim, G = c->group, lanes = c->lanes_per_layer;
  // layout inside the static array: parked logits | split partials, each region 256-byte aligned
  const size_t logit_bytes = (lanes * G * (size_t)c->cap * 4 + 255) & ~(size_t)255;
  const size_t part_bytes = lanes * (size_t)c->n_splits * G * (D + 2) * 4;
  const size_t need = logit_bytes + part_bytes;
  if (need > kStaticScratchBytes)
    return fail(c, WKV_ERR_INVALID,
                "wkv_decode_step_static: this shape needs " + std::to_string(need) + " bytes of scratch, the built-in array holds " +
                    std::to_string(kStaticScratchBytes) + " (WKV_STATIC_SCRATCH_BYTES); use wkv_decode_step");
  unsigned char* base = nullptr;
  cudaError_t e = static_scratch_base(&base);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaGetSymbolAddress(static scratch)");
  wkv::StepParams P = base_params(c, layer);
  P.logits = reinterpret_cast<float*>(base);
  P.part = reinterpret_cast<float*>(base + logit_bytes);
  P.q = q; P.k = k; P.v = v; P.out = out; P.evicted = evicted_pos; P.probs = nullptr;
  P.q_bs = (long long)c->cfg.n_q_heads * (long long)D;
  P.kv_bs = (long long)c->cfg.n_kv_heads * (long long)D;
  P.out_bs = P.q_bs;
  P.ev_bs = c->cfg.n_kv_heads;
  P.seq_lens = nullptr;
  P.tok_idx = 0;
  // The array keeps whatever the previous call (of any context) left.  Nothing in it has to start at zero: the scan
  // kernel writes every logit and every partial of an active lane before the epilogue kernel reads them.
  P.wait_at_start = 2;                 // one array for everybody: never start before the previous kernel has finished
  c->last_layer = -1;
  c->tokens_hi[layer] += 1;
  g_last_launcher.store(nullptr);
  e = launch_any(c, P, false);
  c->launches += 2;
  if (e != cudaSuccess) return cuda_fail(c, e, "decode step launch (static scratch)");
  return WKV_OK;
}

int wkv_decode_step_host(wkv_ctx* c, int32_t layer, const void* q, const void* k, const void* v, void* out,
                         int32_t* evicted_pos) {
  if (!c) return WKV_ERR_INVALID;
  if (!q || !k || !v || !out) return fail(c, WKV_ERR_INVALID, "q, k, v and out must not be NULL");
  const size_t row = (size_t)c->cfg.head_dim * c->elem;
  const size_t qb = (size_t)c->cfg.batch * c->cfg.n_q_heads * row, kb = (size_t)c->lanes_per_layer * row;
  WKV_CUDA(c, cudaMemcpyAsync(c->stage_q, q, qb, cudaMemcpyHostToDevice, c->stream));
  WKV_CUDA(c, cudaMemcpyAsync(c->stage_k, k, kb, cudaMemcpyHostToDevice, c->stream));
  WKV_CUDA(c, cudaMemcpyAsync(c->stage_v, v, kb, cudaMemcpyHostToDevice, c->stream));
  int rc = decode_step_impl(c, layer, c->stage_q, c->stage_k, c->stage_v, c->stage_out, c->stage_ev, nullptr, false);
  if (rc != WKV_OK) return rc;
  WKV_CUDA(c, cudaMemcpyAsync(out, c->stage_out, qb, cudaMemcpyDeviceToHost, c->stream));
  if (evicted_pos)
    WKV_CUDA(c, cudaMemcpyAsync(evicted_pos, c->stage_ev, (size_t)c->lanes_per_layer * 4, cudaMemcpyDeviceToHost, c->stream));
  WKV_CUDA(c, cudaStreamSynchronize(c->stream));
  return WKV_OK;
}

int wkv_decode_step_layers_host(wkv_ctx* c, const void* q, const void* k, const void* v, void* out, int32_t* evicted_pos) {
  if (!c) return WKV_ERR_INVALID;
  if (!q || !k || !v || !out) return fail(c, WKV_ERR_INVALID, "q, k, v and out must not be NULL");
  const size_t row = (size_t)c->cfg.head_dim * c->elem;
  const size_t qb = (size_t)c->cfg.n_layers * c->cfg.batch * c->cfg.n_q_heads * row, kb = (size_t)c->lanes_total * row;
  WKV_CUDA(c, cudaMemcpyAsync(c->stage_q, q, qb, cudaMemcpyHostToDevice, c->stream));
  WKV_CUDA(c, cudaMemcpyAsync(c->stage_k, k, kb, cudaMemcpyHostToDevice, c->stream));
  WKV_CUDA(c, cudaMemcpyAsync(c->stage_v, v, kb, cudaMemcpyHostToDevice, c->stream));
  int rc = wkv_decode_step_layers(c, c->stage_q, c->stage_k, c->stage_v, c->stage_out, c->stage_ev);
  if (rc != WKV_OK) return rc;
  WKV_CUDA(c, cudaMemcpyAsync(out, c->stage_out, qb, cudaMemcpyDeviceToHost, c->stream));
  if (evicted_pos)
    WKV_CUDA(c, cudaMemcpyAsync(evicted_pos, c->stage_ev, (size_t)c->lanes_total * 4, cudaMemcpyDeviceToHost, c->stream));
  WKV_CUDA(c, cudaStreamSynchronize(c->stream));
  return WKV_OK;
}

// Tokens [t_begin, T_max) of a prompt, one step of Algorithm 1 per token.
static int stream_tokens(wkv_ctx* c, int32_t layer, const void* Q, const void* K, const void* V, const int32_t* seq_lens,
                         int32_t t_begin, int32_t T_max, void* out, int32_t* evicted_pos) {
  const long long D = c->cfg.head_dim, Hq = c->cfg.n_q_heads, Hk = c->cfg.n_kv_heads;
  wkv::StepParams P = base_params(c, layer);
  P.seq_lens = seq_lens;
  P.q_bs = (long long)T_max * Hq * D;
  P.kv_bs = (long long)T_max * Hk * D;
  P.out_bs = out ? P.q_bs : Hq * D;
  P.ev_bs = evicted_pos ? (long long)T_max * Hk : Hk;
  if (t_begin < T_max) c->tokens_hi[layer] += T_max - t_begin;
  for (int t = t_begin; t < T_max; ++t) {
    P.tok_idx = t;
    P.q = (const char*)Q + (size_t)t * Hq * D * c->elem;
    P.k = (const char*)K + (size_t)t * Hk * D * c->elem;
    P.v = (const char*)V + (size_t)t * Hk * D * c->elem;
    P.out = out ? (void*)((char*)out + (size_t)t * Hq * D * c->elem) : c->stage_out;
    P.evicted = evicted_pos ? evicted_pos + (size_t)t * Hk : c->stage_ev;
    if (!c->use_cluster) prepare_overlap(c, P, layer, 0, 0, false);     // token after token on one layer: no overlap
    cudaError_t e = launch_any(c, P, c->use_cluster);
    c->launches += c->use_cluster ? 1 : 2;
    if (e != cudaSuccess) return cuda_fail(c, e, "decode step launch (prefill)");
  }
  note_outputs(c, nullptr, 0, nullptr, 0, nullptr, 0);
  return WKV_OK;
}

}  // extern "C"

// ---- blocked prompt tail (wkv_block.cuh) --------------------------------------------------------------------------
// Tokens per block for this context, or 0 where the tail is streamed token by token: the block's query rows (tokens x
// query heads per key) must be 8 at most, the window must be longer than the block (an entry removed inside the block and
// its right neighbour are then never tokens of the block), and the lane epilogue must be the register version.
static int block_tokens_of(const wkv_ctx* c, int lanes) {
  if (c->group > 4) return 0;
  const int B = 8 / c->group;
  if (c->cfg.window <= B) return 0;
  const int nt = epilogue_threads(c->group, lanes, c->sm_count);
  if (c->cfg.budget + 1 > wkv::epilogue_slots_per_thread(c->group, nt) * nt) return 0;
  return B;
}

// Scratch of the blocked tail for `lanes` lanes, taken from the provider on first use (or when more lanes are needed).
// false: the provider refused; the caller then streams the tokens instead -- nothing has been launched for them yet.
static bool block_scratch(wkv_ctx* c, int lanes, int B) {
  if (c->blk_logits != nullptr && c->blk_lanes >= lanes) return true;
  const size_t cap = c->cap, D = c->cfg.head_dim;
  const int R = 8;
  const int tiles = (c->cfg.budget + 1 + wkv::kTileSlots - 1) / wkv::kTileSlots;
  int units = (int)((6LL * c->sm_count + lanes - 1) / lanes);
  units = std::max(1, std::min({units, 16, std::max(1, tiles / 8)}));
  int rc = take(c, &c->blk_logits, (size_t)lanes * R * cap * 4);
  if (rc == WKV_OK) rc = take(c, &c->blk_lgx, (size_t)lanes * R * B * 4 + 256);
  if (rc == WKV_OK) rc = take(c, &c->blk_ptab, (size_t)lanes * R * cap * 4 + 256);   // the last tile of the last row is read whole
  if (rc == WKV_OK) rc = take(c, &c->blk_opart, (size_t)lanes * units * R * D * 4);
  if (rc == WKV_OK) rc = take(c, &c->blk_rec_rows, (size_t)lanes * 2 * B * D * 4);
  if (rc == WKV_OK) rc = take(c, &c->blk_rec_slot, (size_t)lanes * 2 * B * 4);
  if (rc != WKV_OK) { c->blk_logits = nullptr; c->blk_lanes = 0; return false; }
  c->blk_lanes = lanes;
  c->blk_units = units;
  return true;
}

template <typename T, int D>
static cudaError_t launch_block_kernels(int which, const wkv::BlockParams& BP, int lanes, cudaStream_t s) {
  using namespace wkv;
  constexpr int R = 8;
  if (which == 0) {
    constexpr int smem = BlockCfg<T, D, R>::kLogitsSmem;
    cudaError_t e = cudaFuncSetAttribute(block_logits_kernel<T, D, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    block_logits_kernel<T, D, R><<<lanes * BP.n_units, kThreads, smem, s>>>(BP);
  } else if (which == 1) {
    constexpr int smem = BlockCfg<T, D, R>::kPvSmem;
    constexpr bool mma = BlockCfg<T, D, R>::kPvMma;      // bf16 rows: on the tensor cores
    cudaError_t e = cudaFuncSetAttribute(block_pv_kernel<T, D, R, mma>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    block_pv_kernel<T, D, R, mma><<<lanes * BP.n_units, kThreads, smem, s>>>(BP);
  } else {
    block_out_kernel<T, D><<<lanes * BP.block_tokens * BP.group, D, 0, s>>>(BP);
  }
  return cudaGetLastError();
}
static cudaError_t launch_block(const wkv_ctx* c, int which, const wkv::BlockParams& BP, int lanes) {
  if (c->cfg.dtype == WKV_BF16)
    return c->cfg.head_dim == 128 ? launch_block_kernels<__nv_bfloat16, 128>(which, BP, lanes, c->stream)
                                  : launch_block_kernels<__nv_bfloat16, 64>(which, BP, lanes, c->stream);
  return c->cfg.head_dim == 128 ? launch_block_kernels<float, 128>(which, BP, lanes, c->stream)
                                : launch_block_kernels<float, 64>(which, BP, lanes, c->stream);
}
template <typename T, int D>
static cudaError_t launch_epilogue_by_group(int G, const wkv::StepParams& P, int lanes, int dev, cudaStream_t s) {
  switch (G) {
    case 1: return launch_epilogue<T, D, 1>(P, lanes, dev, s, true);
    case 2: return launch_epilogue<T, D, 2>(P, lanes, dev, s, true);
    case 4: return launch_epilogue<T, D, 4>(P, lanes, dev, s, true);
  }
  return cudaErrorInvalidValue;
}
static cudaError_t launch_epilogue_any(const wkv_ctx* c, const wkv::StepParams& P, int lanes) {
  if (c->cfg.dtype == WKV_BF16)
    return c->cfg.head_dim == 128 ? launch_epilogue_by_group<__nv_bfloat16, 128>(c->group, P, lanes, c->device, c->stream)
                                  : launch_epilogue_by_group<__nv_bfloat16, 64>(c->group, P, lanes, c->device, c->stream);
  return c->cfg.head_dim == 128 ? launch_epilogue_by_group<float, 128>(c->group, P, lanes, c->device, c->stream)
                                : launch_epilogue_by_group<float, 64>(c->group, P, lanes, c->device, c->stream);
}

// Tokens [t_begin, T_max) of a prompt for `lanes` consecutive lanes starting at lane0 (one layer, or all layers: to the
// kernels the sequences of several layers are just more sequences), B tokens per pair of cache sweeps.
// q_bs / kv_bs: batch strides of Q and K, V in elements; seq_lens indexed by lane / n_kv_heads.
static int blocked_tokens(wkv_ctx* c, long long lane0, int lanes, int B, const void* Q, const void* K, const void* V,
                          const int32_t* seq_lens, int32_t t_begin, int32_t T_max, void* out, int32_t* evicted_pos) {
  const long long D = c->cfg.head_dim, Hq = c->cfg.n_q_heads, Hk = c->cfg.n_kv_heads;
  const int R = 8, G = c->group;
  const size_t cap = c->cap;
  if (!block_scratch(c, lanes, B)) return WKV_ERR_ALLOC;
  wkv::BlockParams BP;
  std::memset(&BP, 0, sizeof(BP));
  BP.Kc = c->Kc; BP.Vc = c->Vc; BP.lane_state = c->lane_state;
  BP.Q = Q; BP.K = K; BP.out = out; BP.seq_lens = seq_lens;
  BP.logits = c->blk_logits; BP.lgx = c->blk_lgx; BP.ptab = c->blk_ptab; BP.opart = c->blk_opart;
  BP.rec_rows = c->blk_rec_rows; BP.rec_slot = c->blk_rec_slot; BP.status = c->status;
  BP.q_bs = (long long)T_max * Hq * D; BP.kv_bs = (long long)T_max * Hk * D; BP.out_bs = BP.q_bs;
  BP.q_ts = Hq * D; BP.kv_ts = Hk * D; BP.out_ts = Hq * D;
  BP.lane0 = (int)lane0; BP.n_kv_heads = c->cfg.n_kv_heads; BP.cap = c->cap; BP.budget = c->cfg.budget;
  BP.block_tokens = B; BP.group = G; BP.n_units = c->blk_units; BP.scale = c->scale;
  std::memcpy(BP.vmap, c->vmap, sizeof(BP.vmap));

  wkv::StepParams P = base_params(c, 0);
  P.lane0 = (int)lane0;
  P.n_lanes = lanes;
  P.flat_chunk = 0;
  P.n_splits = 1;
  P.part = nullptr;
  P.ticket = nullptr;
  P.wait_at_start = 2;
  P.logits = c->blk_logits;
  P.lgx = c->blk_lgx;
  P.rec_rows = c->blk_rec_rows;
  P.rec_slot = c->blk_rec_slot;
  P.logit_rows = R;
  P.block_tokens = B;
  P.probs = out ? c->blk_ptab : nullptr;
  P.probs_rows = R;
  P.probs_stride = (int)cap;
  P.seq_lens = seq_lens;
  P.q_bs = BP.q_bs; P.kv_bs = BP.kv_bs;
  P.out = nullptr; P.out_bs = 0;
  P.ev_bs = evicted_pos ? (long long)T_max * Hk : Hk;
  for (int t0 = t_begin; t0 < T_max; t0 += B) {
    const int n_tok = std::min<int>(B, T_max - t0);
    BP.tok0 = t0;
    BP.n_tok = n_tok;
    cudaError_t e = launch_block(c, 0, BP, lanes);
    c->launches += 1;
    if (e != cudaSuccess) return cuda_fail(c, e, "block logits launch");
    // the block's tokens, one after the other inside one launch
    P.tok_idx = t0;
    P.block_n = n_tok;
    P.k = (const char*)K + (size_t)t0 * Hk * D * c->elem;
    P.v = (const char*)V + (size_t)t0 * Hk * D * c->elem;
    P.kv_ts = Hk * D;
    P.evicted = evicted_pos ? evicted_pos + (size_t)t0 * Hk : c->stage_ev;
    P.ev_ts = evicted_pos ? Hk : 0;
    e = launch_epilogue_any(c, P, lanes);
    c->launches += 1;
    if (e != cudaSuccess) return cuda_fail(c, e, "lane epilogue launch (blocked prompt tail)");
    if (out) {
      e = launch_block(c, 1, BP, lanes);
      if (e == cudaSuccess) e = launch_block(c, 2, BP, lanes);
      c->launches += 2;
      if (e != cudaSuccess) return cuda_fail(c, e, "block output launch");
    }
  }
  c->last_layer = -1;
  g_last_launcher.store(nullptr);
  note_outputs(c, nullptr, 0, nullptr, 0, nullptr, 0);
  return WKV_OK;
}

extern "C" {

static int check_prefill_args(wkv_ctx* c, int32_t layer, const void* Q, const void* K, const void* V, int32_t T_max) {
  if (!c) return WKV_ERR_INVALID;
  if (!Q || !K || !V) return fail(c, WKV_ERR_INVALID, "Q, K and V must not be NULL");
  if (layer < 0 || layer >= c->cfg.n_layers) return fail(c, WKV_ERR_INVALID, "layer out of range");
  if (T_max < 0) return fail(c, WKV_ERR_INVALID, "T_max must be >= 0");
  return WKV_OK;
}

int wkv_prefill(wkv_ctx* c, int32_t layer, const void* Q, const void* K, const void* V, const int32_t* seq_lens,
                int32_t T_max, void* out, int32_t* evicted_pos) {
  const int rc = check_prefill_args(c, layer, Q, K, V, T_max);
  if (rc != WKV_OK) return rc;
  return stream_tokens(c, layer, Q, K, V, seq_lens, 0, T_max, out, evicted_pos);
}

// The dense kernel over `lanes` consecutive lanes starting at lane0 (one layer, or all layers at once: to the kernel the
// lanes of several layers are just more sequences).  Takes the scratch on first use / when more lanes are needed.
// Which geometry the dense prompt kernel runs with for a launch of `lanes` lanes: blocks of 32 query rows (256 threads,
// two CTAs per SM) while two CTAs per SM hold every lane, else blocks of 16 rows (128 threads, four CTAs per SM).
static bool dense_rows_wide(const wkv_ctx* c, long long lanes) {
  return c->cfg.dtype == WKV_BF16 && lanes <= 2LL * c->sm_count;
}
static int launch_dense(wkv_ctx* c, long long lane0, long long lanes, const void* Q, const void* K, const void* V,
                        const int32_t* seq_lens, int32_t T_max, int32_t n0, void* out, int32_t* evicted_pos) {
  // few lanes (at most two per SM): blocks of 32 query rows on 256 threads; else 16 rows on 128 threads, four CTAs per SM
  const bool wide = dense_rows_wide(c, lanes);
  const int rows = wide ? wkv::kBulkRowsWide : wkv::kBulkRows;
  if (c->bulk_S == nullptr || c->bulk_lanes * c->bulk_rows < lanes * rows) {
    c->bulk_stride = (c->cfg.budget + wkv::kBulkKeys - 1) / wkv::kBulkKeys * wkv::kBulkKeys;
    int rc = take(c, &c->bulk_S, (size_t)lanes * rows * c->bulk_stride * 4);
    if (rc != WKV_OK) return rc;
    c->bulk_lanes = lanes;
    c->bulk_rows = rows;
  }
  wkv::PrefillParams P;
  std::memset(&P, 0, sizeof(P));
  P.Kc = c->Kc; P.Vc = c->Vc; P.a = c->a; P.pos = c->pos; P.next = c->next; P.prev = c->prev;
  P.lane_state = c->lane_state;
  P.S = c->bulk_S;
  P.Q = Q; P.K = K; P.V = V; P.out = out; P.evicted = evicted_pos; P.seq_lens = seq_lens;
  P.batch = c->cfg.batch;
  P.lane0 = (int)lane0;
  P.n_kv_heads = c->cfg.n_kv_heads;
  P.cap = c->cap;
  P.T_max = T_max;
  P.n0 = n0;
  P.s_stride = c->bulk_stride;
  P.scale = c->scale;
  P.status = c->status;
  cudaError_t e;
  const int n = (int)lanes;
  if (c->cfg.dtype == WKV_BF16) {
    // the kernel takes its tiles through the tensor maps over the caches (boxes of one tile of 64 keys)
    std::memcpy(P.kmap, c->dense_kmap, sizeof(P.kmap));
    std::memcpy(P.vmap, c->dense_vmap, sizeof(P.vmap));
    if (wide)
      e = c->cfg.head_dim == 128 ? launch_bulk<__nv_bfloat16, 128, 64, wkv::kBulkRowsWide>(c->group, P, n, c->stream)
                                 : launch_bulk<__nv_bfloat16, 64, 64, wkv::kBulkRowsWide>(c->group, P, n, c->stream);
    else
      e = c->cfg.head_dim == 128 ? launch_bulk<__nv_bfloat16, 128, 64>(c->group, P, n, c->stream)
                                 : launch_bulk<__nv_bfloat16, 64, 64>(c->group, P, n, c->stream);
  } else {
    e = c->cfg.head_dim == 128 ? launch_bulk<float, 128, 64>(c->group, P, n, c->stream)
                               : launch_bulk<float, 64, 64>(c->group, P, n, c->stream);
  }
  c->launches += 1;
  if (e != cudaSuccess) return cuda_fail(c, e, "bulk prefill launch");
  c->last_layer = -1;                    // the next scan of this context waits for this kernel before anything else
  g_last_launcher.store(nullptr);
  note_outputs(c, nullptr, 0, nullptr, 0, nullptr, 0);
  return WKV_OK;
}

int wkv_prefill_bulk(wkv_ctx* c, int32_t layer, const void* Q, const void* K, const void* V, const int32_t* seq_lens,
                     int32_t T_max, void* out, int32_t* evicted_pos) {
  int rc = check_prefill_args(c, layer, Q, K, V, T_max);
  if (rc != WKV_OK) return rc;
  // the dense kernel moves rows with 16-byte bulk copies and vector loads / stores
  if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)out) & 15)
    return fail(c, WKV_ERR_INVALID, "wkv_prefill_bulk: Q, K, V and out must be 16-byte aligned");
  int32_t n0 = 0;
  const long long room = (long long)c->cfg.budget - c->tokens_hi[layer];
  if (room > 0 && T_max > 0) {
    // No lane of the layer can hold more than budget - room tokens, so none has compressed and the next `room` tokens
    // compress nothing either: the first min(T_max, room) tokens of this call go through the dense kernel (on top of
    // whatever each lane already holds), the rest is streamed behind it on the same stream.
    n0 = (int32_t)std::min<long long>(T_max, room);
    rc = launch_dense(c, (long long)layer * c->lanes_per_layer, c->lanes_per_layer, Q, K, V, seq_lens, T_max, n0, out,
                      evicted_pos);
    if (rc != WKV_OK) return rc;
    c->tokens_hi[layer] += n0;
  }
  // the rest: in blocks of tokens that share two sweeps of the cache where the configuration allows, else token by token
  const int B = block_tokens_of(c, c->lanes_per_layer);
  if (B > 0 && T_max - n0 >= 2 && block_scratch(c, c->lanes_per_layer, B)) {
    c->tokens_hi[layer] += T_max - n0;
    return blocked_tokens(c, (long long)layer * c->lanes_per_layer, c->lanes_per_layer, B, Q, K, V, seq_lens, n0, T_max, out,
                          evicted_pos);
  }
  return stream_tokens(c, layer, Q, K, V, seq_lens, n0, T_max, out, evicted_pos);
}

int wkv_prefill_bulk_layers(wkv_ctx* c, const void* Q, const void* K, const void* V, const int32_t* seq_lens,
                            int32_t T_max, void* out, int32_t* evicted_pos) {
  int rc = check_prefill_args(c, 0, Q, K, V, T_max);
  if (rc != WKV_OK) return rc;
  if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)out) & 15)
    return fail(c, WKV_ERR_INVALID, "wkv_prefill_bulk_layers: Q, K, V and out must be 16-byte aligned");
  const long long D = c->cfg.head_dim, Hq = c->cfg.n_q_heads, Hk = c->cfg.n_kv_heads, B = c->cfg.batch;
  const int L = c->cfg.n_layers;
  const size_t q_layer = (size_t)B * T_max * Hq * D * c->elem, kv_layer = (size_t)B * T_max * Hk * D * c->elem;
  const size_t ev_layer = (size_t)B * T_max * Hk;
  if (ranges_overlap(Q, q_layer * L, out, q_layer * L) || ranges_overlap(K, kv_layer * L, out, q_layer * L) ||
      ranges_overlap(V, kv_layer * L, out, q_layer * L) || ranges_overlap(Q, q_layer * L, evicted_pos, ev_layer * 4 * L) ||
      ranges_overlap(K, kv_layer * L, evicted_pos, ev_layer * 4 * L) || ranges_overlap(V, kv_layer * L, evicted_pos, ev_layer * 4 * L))
    return fail(c, WKV_ERR_INVALID, "wkv_prefill_bulk_layers: inputs and outputs must not overlap");
  long long room = c->cfg.budget;
  for (int l = 0; l < L; ++l) room = std::min(room, (long long)c->cfg.budget - c->tokens_hi[l]);
  int32_t n0 = 0;
  if (room > 0 && T_max > 0) {
    n0 = (int32_t)std::min<long long>(T_max, room);        // uncompressed in every lane of every layer (see wkv_prefill_bulk)
    const int stride = (c->cfg.budget + wkv::kBulkKeys - 1) / wkv::kBulkKeys * wkv::kBulkKeys;
    const size_t need_all = (size_t)c->lanes_total * (dense_rows_wide(c, c->lanes_total) ? wkv::kBulkRowsWide : wkv::kBulkRows) * stride * 4;
    if (need_all <= ((size_t)256 << 20)) {
      // every lane of every layer in one launch
      rc = launch_dense(c, 0, c->lanes_total, Q, K, V, seq_lens, T_max, n0, out, evicted_pos);
      if (rc != WKV_OK) return rc;
    } else {
      for (int l = 0; l < L; ++l) {
        rc = launch_dense(c, (long long)l * c->lanes_per_layer, c->lanes_per_layer, (const char*)Q + l * q_layer,
                          (const char*)K + l * kv_layer, (const char*)V + l * kv_layer, seq_lens, T_max, n0,
                          out ? (char*)out + l * q_layer : nullptr, evicted_pos ? evicted_pos + l * ev_layer : nullptr);
        if (rc != WKV_OK) return rc;
      }
    }
    for (auto& th : c->tokens_hi) th += n0;
  }
  // The rest of the prompt, token by token with the layers interleaved: consecutive launches then belong to different
  // layers, and since every input of this call existed before it was issued, a layer's scan may overlap the previous
  // layer's lane epilogues.
  for (auto& th : c->tokens_hi) th += T_max - n0;
  c->last_layer = -1;
  if (T_max - n0 >= 2) {
    // the rest in blocks of tokens (wkv_block.cuh) where the configuration allows: over the lanes of all layers at once
    // when a layer alone is small, else layer after layer (the layers' prompts are independent)
    const int B_all = c->fused_ok ? block_tokens_of(c, (int)c->lanes_total) : 0;
    const int B_one = block_tokens_of(c, c->lanes_per_layer);
    if (B_all > 0 && block_scratch(c, (int)c->lanes_total, B_all)) {
      if (seq_lens != nullptr)
        for (int l = 0; l < L; ++l)
          WKV_CUDA(c, cudaMemcpyAsync(c->fused_seq_lens + (size_t)l * B, seq_lens, (size_t)B * 4, cudaMemcpyDeviceToDevice, c->stream));
      return blocked_tokens(c, 0, (int)c->lanes_total, B_all, Q, K, V, seq_lens != nullptr ? c->fused_seq_lens : nullptr, n0, T_max,
                            out, evicted_pos);
    }
    if (B_one > 0 && block_scratch(c, c->lanes_per_layer, B_one)) {
      for (int l = 0; l < L; ++l) {
        rc = blocked_tokens(c, (long long)l * c->lanes_per_layer, c->lanes_per_layer, B_one, (const char*)Q + l * q_layer,
                            (const char*)K + l * kv_layer, (const char*)V + l * kv_layer, seq_lens, n0, T_max,
                            out ? (char*)out + l * q_layer : nullptr, evicted_pos ? evicted_pos + l * ev_layer : nullptr);
        if (rc != WKV_OK) return rc;
      }
      return WKV_OK;
    }
  }
  if (c->fused_ok && n0 < T_max) {
    // a layer alone cannot fill the GPU: one launch (pair) per token over the lanes of all layers, as in
    // wkv_decode_step_layers; [n_layers, batch, ...] is [n_layers * batch, ...] to the kernels
    if (seq_lens != nullptr)
      for (int l = 0; l < L; ++l)
        WKV_CUDA(c, cudaMemcpyAsync(c->fused_seq_lens + (size_t)l * B, seq_lens, (size_t)B * 4, cudaMemcpyDeviceToDevice, c->stream));
    wkv::StepParams P = base_params(c, 0);
    P.n_splits = c->fused_splits;
    P.flat_chunk = c->fused_flat_chunk;
    P.chunk_cap = c->fused_chunk_cap;
    P.logits = c->fused_logits;
    P.part = c->fused_part;
    P.ticket = c->fused_ticket;
    P.seq_lens = seq_lens != nullptr ? c->fused_seq_lens : nullptr;
    P.q_bs = (long long)T_max * Hq * D;
    P.kv_bs = (long long)T_max * Hk * D;
    P.out_bs = out ? P.q_bs : Hq * D;
    P.ev_bs = evicted_pos ? (long long)T_max * Hk : Hk;
    P.wait_at_start = 2;
    g_last_launcher.store(c);
    for (int t = n0; t < T_max; ++t) {
      P.tok_idx = t;
      P.q = (const char*)Q + (size_t)t * Hq * D * c->elem;
      P.k = (const char*)K + (size_t)t * Hk * D * c->elem;
      P.v = (const char*)V + (size_t)t * Hk * D * c->elem;
      P.out = out ? (void*)((char*)out + (size_t)t * Hq * D * c->elem) : c->stage_out;
      P.evicted = evicted_pos ? evicted_pos + (size_t)t * Hk : c->stage_ev;
      cudaError_t e = launch_any(c, P, c->fused_cluster, (int)c->lanes_total);
      c->launches += c->fused_cluster ? 1 : 2;
      if (e != cudaSuccess) return cuda_fail(c, e, "decode step launch (prefill, all layers at once)");
    }
    note_outputs(c, nullptr, 0, nullptr, 0, nullptr, 0);
    return WKV_OK;
  }
  for (int t = n0; t < T_max; ++t) {
    for (int l = 0; l < L; ++l) {
      wkv::StepParams P = base_params(c, l);
      P.seq_lens = seq_lens;
      P.q_bs = (long long)T_max * Hq * D;
      P.kv_bs = (long long)T_max * Hk * D;
      P.out_bs = out ? P.q_bs : Hq * D;
      P.ev_bs = evicted_pos ? (long long)T_max * Hk : Hk;
      P.tok_idx = t;
      P.q = (const char*)Q + l * q_layer + (size_t)t * Hq * D * c->elem;
      P.k = (const char*)K + l * kv_layer + (size_t)t * Hk * D * c->elem;
      P.v = (const char*)V + l * kv_layer + (size_t)t * Hk * D * c->elem;
      P.out = out ? (void*)((char*)out + l * q_layer + (size_t)t * Hq * D * c->elem)
                  : (void*)((char*)c->stage_out + (size_t)l * B * Hq * D * c->elem);
      P.evicted = evicted_pos ? evicted_pos + l * ev_layer + (size_t)t * Hk : c->stage_ev + (size_t)l * c->lanes_per_layer;
      // As in wkv_decode_step_layers, the first layer of every token waits for everything before it (the same lanes
      // were written one token ago); the layers behind it start once its units are in scratch, hence after that wait.
      if (l == 0) c->last_layer = -1;
      if (!c->use_cluster) prepare_overlap(c, P, l, 0, 0, true);
      cudaError_t e = launch_any(c, P, c->use_cluster);
      c->launches += c->use_cluster ? 1 : 2;
      if (e != cudaSuccess) return cuda_fail(c, e, "decode step launch (prefill, all layers)");
    }
  }
  c->last_layer = -1;
  note_outputs(c, nullptr, 0, nullptr, 0, nullptr, 0);
  return WKV_OK;
}

int wkv_export_state(wkv_ctx* c, int32_t layer, int32_t b, int32_t kv_head, int32_t* len, int32_t* tokens, int32_t* pos,
                     float* a, void* K, void* V) {
  int rc = check_lane(c, layer, b, kv_head);
  if (rc != WKV_OK) return rc;
  const long long lane = ((long long)layer * c->cfg.batch + b) * c->cfg.n_kv_heads + kv_head;
  const int cap = c->cap, D = c->cfg.head_dim;
  const size_t row = (size_t)D * c->elem;
  int32_t st[wkv::LS_STRIDE];
  std::vector<int32_t> hpos(cap), hnext(cap), hprev(cap);
  std::vector<float> ha(cap);
  std::vector<char> hK, hV;
  WKV_CUDA(c, cudaStreamSynchronize(c->stream));
  WKV_CUDA(c, cudaMemcpy(st, c->lane_state + lane * wkv::LS_STRIDE, sizeof(st), cudaMemcpyDeviceToHost));
  WKV_CUDA(c, cudaMemcpy(hpos.data(), c->pos + lane * cap, cap * 4, cudaMemcpyDeviceToHost));
  WKV_CUDA(c, cudaMemcpy(hnext.data(), c->next + lane * cap, cap * 4, cudaMemcpyDeviceToHost));
  WKV_CUDA(c, cudaMemcpy(hprev.data(), c->prev + lane * cap, cap * 4, cudaMemcpyDeviceToHost));
  WKV_CUDA(c, cudaMemcpy(ha.data(), c->a + lane * cap, cap * 4, cudaMemcpyDeviceToHost));
  if (K) { hK.resize(cap * row); WKV_CUDA(c, cudaMemcpy(hK.data(), (char*)c->Kc + lane * cap * row, cap * row, cudaMemcpyDeviceToHost)); }
  if (V) { hV.resize(cap * row); WKV_CUDA(c, cudaMemcpy(hV.data(), (char*)c->Vc + lane * cap * row, cap * row, cudaMemcpyDeviceToHost)); }
  const int n = st[wkv::LS_LEN];
  if (n < 0 || n > c->cfg.budget) return fail(c, WKV_ERR_STATE, "lane length out of range");
  if (len) *len = n;
  if (tokens) *tokens = st[wkv::LS_T];
  // walk the chain: exactly n entries, consistent back links, strictly increasing positions
  int s = st[wkv::LS_HEAD], prev_slot = -1, last_pos = -1;
  for (int i = 0; i < n; ++i) {
    if (s < 0 || s >= cap) return fail(c, WKV_ERR_STATE, "chain leaves the slot range");
    if (hprev[s] != prev_slot) return fail(c, WKV_ERR_STATE, "back link does not match");
    if (hpos[s] <= last_pos || hpos[s] >= st[wkv::LS_T]) return fail(c, WKV_ERR_STATE, "positions not strictly increasing");
    if (pos) pos[i] = hpos[s];
    if (a) a[i] = ha[s];
    if (K) std::memcpy((char*)K + i * row, hK.data() + s * row, row);
    if (V) std::memcpy((char*)V + i * row, hV.data() + s * row, row);
    last_pos = hpos[s];
    prev_slot = s;
    s = hnext[s];
  }
  if (n > 0 && (s != -1 || prev_slot != st[wkv::LS_TAIL])) return fail(c, WKV_ERR_STATE, "chain does not end at the tail");
  if (n == 0 && st[wkv::LS_HEAD] != -1) return fail(c, WKV_ERR_STATE, "empty lane with a head");
  return WKV_OK;
}

int wkv_export_slots(wkv_ctx* c, int32_t layer, int32_t b, int32_t kv_head, int32_t* slot_pos) {
  int rc = check_lane(c, layer, b, kv_head);
  if (rc != WKV_OK) return rc;
  if (!slot_pos) return fail(c, WKV_ERR_INVALID, "slot_pos must not be NULL");
  const long long lane = ((long long)layer * c->cfg.batch + b) * c->cfg.n_kv_heads + kv_head;
  WKV_CUDA(c, cudaStreamSynchronize(c->stream));
  WKV_CUDA(c, cudaMemcpy(slot_pos, c->pos + lane * c->cap, (size_t)(c->cfg.budget + 1) * 4, cudaMemcpyDeviceToHost));
  return WKV_OK;
}

int wkv_import_state(wkv_ctx* c, int32_t layer, int32_t b, int32_t kv_head, int32_t len, int32_t tokens,
                     const int32_t* pos, const float* a, const void* K, const void* V) {
  int rc = check_lane(c, layer, b, kv_head);
  if (rc != WKV_OK) return rc;
  if (len < 0 || len > c->cfg.budget || tokens < len) return fail(c, WKV_ERR_INVALID, "len / tokens out of range");
  if (len > 0 && (!pos || !a || !K || !V)) return fail(c, WKV_ERR_INVALID, "pos, a, K, V must not be NULL");
  for (int i = 0; i < len; ++i)
    if (pos[i] < 0 || pos[i] >= tokens || (i > 0 && pos[i] <= pos[i - 1]))
      return fail(c, WKV_ERR_INVALID, "pos must be strictly increasing and < tokens");
  const long long lane = ((long long)layer * c->cfg.batch + b) * c->cfg.n_kv_heads + kv_head;
  const int cap = c->cap;
  const size_t row = (size_t)c->cfg.head_dim * c->elem;
  // an imported lane counts as uncompressed only if it is: every token still there, hence token i in slot i
  c->tokens_hi[layer] = tokens == len ? std::max<long long>(c->tokens_hi[layer], tokens) : (long long)c->cfg.budget;
  std::vector<int32_t> hpos(cap, -1), hnext(cap, -1), hprev(cap, -1);
  std::vector<float> ha(cap, 0.f);
  for (int i = 0; i < len; ++i) {
    hpos[i] = pos[i];
    ha[i] = a[i];
    hnext[i] = i + 1 < len ? i + 1 : -1;
    hprev[i] = i - 1;
  }
  int32_t st[wkv::LS_STRIDE] = {len, tokens, len > 0 ? 0 : -1, len > 0 ? len - 1 : -1, len, 0, 0, 0};
  WKV_CUDA(c, cudaStreamSynchronize(c->stream));
  WKV_CUDA(c, cudaMemcpy(c->pos + lane * cap, hpos.data(), cap * 4, cudaMemcpyHostToDevice));
  WKV_CUDA(c, cudaMemcpy(c->next + lane * cap, hnext.data(), cap * 4, cudaMemcpyHostToDevice));
  WKV_CUDA(c, cudaMemcpy(c->prev + lane * cap, hprev.data(), cap * 4, cudaMemcpyHostToDevice));
  WKV_CUDA(c, cudaMemcpy(c->a + lane * cap, ha.data(), cap * 4, cudaMemcpyHostToDevice));
  if (len > 0) {
    WKV_CUDA(c, cudaMemcpy((char*)c->Kc + lane * cap * row, K, len * row, cudaMemcpyHostToDevice));
    WKV_CUDA(c, cudaMemcpy((char*)c->Vc + lane * cap * row, V, len * row, cudaMemcpyHostToDevice));
  }
  WKV_CUDA(c, cudaMemcpy(c->lane_state + lane * wkv::LS_STRIDE, st, sizeof(st), cudaMemcpyHostToDevice));
  return WKV_OK;
}

int wkv_status(wkv_ctx* c) {
  if (!c) return WKV_ERR_INVALID;
  uint32_t w = 0;
  WKV_CUDA(c, cudaStreamSynchronize(c->stream));
  WKV_CUDA(c, cudaMemcpy(&w, c->status, 4, cudaMemcpyDeviceToHost));
  if (w) {
    WKV_CUDA(c, cudaMemset(c->status, 0, 4));
    if (w & wkv::kStatusWaitTimeout) {
      // A lane epilogue that gave up on its units left their reports uncounted: clear the counters (the stream is
      // idle), so that the next call's epilogues wait for that call's units and not for stale ones.  The lanes that were
      // skipped are one token behind; the caller resets or re-imports them (see wkv.h).
      for (int i = 0; i < 2; ++i) WKV_CUDA(c, cudaMemset(c->ticket[i], 0, (size_t)c->lanes_per_layer * 4));
      if (c->fused_ticket) WKV_CUDA(c, cudaMemset(c->fused_ticket, 0, (size_t)c->lanes_total * 4));
      c->last_layer = -1;
      return fail(c, WKV_ERR_TIMEOUT, "a bounded wait inside a kernel gave up");
    }
    return fail(c, WKV_ERR_STATE, "a kernel found inconsistent slot links");
  }
  return WKV_OK;
}

int wkv_selftest_wait_timeout(wkv_ctx* c) {
  if (!c) return WKV_ERR_INVALID;
  wkv::wait_selftest_kernel<<<1, 32, 0, c->stream>>>(c->status, 20000u);
  c->launches++;
  c->last_layer = -1;
  WKV_CUDA(c, cudaGetLastError());
  return WKV_OK;
}

int64_t wkv_launch_count(const wkv_ctx* c) { return c ? c->launches : 0; }
int64_t wkv_device_bytes(const wkv_ctx* c) { return c ? c->device_bytes : 0; }
int32_t wkv_splits(const wkv_ctx* c) { return c ? c->n_splits : 0; }

const char* wkv_strerror(int code) {
  switch (code) {
    case WKV_OK: return "ok";
    case WKV_ERR_INVALID: return "invalid configuration or argument";
    case WKV_ERR_ALLOC: return "device memory provider failed";
    case WKV_ERR_CUDA: return "CUDA runtime error";
    case WKV_ERR_STATE: return "inconsistent lane bookkeeping";
    case WKV_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown error";
}

const char* wkv_last_error(const wkv_ctx* c) { return c ? c->last_error.c_str() : ""; }

}  // extern "C"
