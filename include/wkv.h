/* wkv.h -- C ABI of the WeightedKV decode hot path for NVIDIA B200 (sm_100a).
 *
 * The library keeps, for every lane = (layer, sequence, kv-head), a key/value cache of at most
 * `budget` entries and runs one iteration of the paper's Algorithm 1 ("WeightedKV") per incoming
 * token: append k_t, v_t; single-query softmax attention over the cache (Background section:
 * A_t = softmax(q_t^T K_t), o_t = A_t^T V_t); fold A_t into the accumulated scores a; once the cache
 * holds more than `budget` entries, pick the entry with the smallest average score a/n outside the
 * protected regions, merge its value into the right neighbour by the score-weighted convex
 * combination, and drop its key.  Lanes are independent (the paper omits the batch and head
 * dimensions for that reason).  Every step of that path runs in CUDA kernels of this library; there
 * is no CPU fallback.
 *
 * Conventions
 *   - "device" pointers are CUDA device addresses on the context's GPU; "host" pointers are ordinary
 *     (preferably page-locked) host addresses.  The library never takes ownership of caller buffers.
 *   - q, k, v, out hold elements of the context's storage type (fp32 or bf16); scores are fp32.
 *   - All calls on one context must be issued from one host thread at a time and run on the
 *     context's stream; device-pointer calls are asynchronous with respect to the host.
 *   - Every function returning int returns WKV_OK (0) or a negative wkv_error; no exceptions cross the
 *     boundary.  wkv_last_error() gives a text for the most recent failure on that context.
 */
#ifndef WKV_H_
#define WKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct wkv_ctx wkv_ctx; /* opaque, library-owned */

typedef enum { WKV_F32 = 0, WKV_BF16 = 1 } wkv_dtype;

typedef enum {
  WKV_OK = 0,
  WKV_ERR_INVALID = -1, /* bad configuration or argument                                   */
  WKV_ERR_ALLOC = -2,   /* the memory provider returned NULL                               */
  WKV_ERR_CUDA = -3,    /* a CUDA runtime call or launch failed (text in wkv_last_error)    */
  WKV_ERR_STATE = -4,   /* a lane's bookkeeping found inconsistent (host check of an export,
                           or a kernel's own check of its slot links)                       */
  WKV_ERR_TIMEOUT = -5  /* a bounded device-side wait gave up (device status word)          */
} wkv_error;

typedef enum {
  WKV_SCHEDULE_AUTO = 0,
  WKV_SCHEDULE_SPLIT = 1,  /* two launches: scan every unit, then one CTA per lane finishes it (any n_splits)    */
  WKV_SCHEDULE_CLUSTER = 2,/* one launch: a lane's units form a thread-block cluster (n_splits in {1,2,4,8,16})  */
  WKV_SCHEDULE_FLAT = 3    /* two launches as in SPLIT, but the scan's CTAs take equal runs of the 32-entry tiles of
                              ALL lanes, across lane boundaries (n_splits = CTAs per lane on average, 0 = one wave
                              that fills the GPU); same results                                                  */
} wkv_schedule;

/* Device memory provider.  alloc returns a device address aligned to at least 256 bytes, or NULL. */
typedef void* (*wkv_alloc_fn)(size_t bytes, void* user);
typedef void (*wkv_release_fn)(void* ptr, void* user);

typedef struct {
  int32_t n_layers;   /* >= 1                                                                          */
  int32_t batch;      /* sequences per call, >= 1                                                      */
  int32_t n_q_heads;  /* query heads; a multiple of n_kv_heads; group = n_q_heads/n_kv_heads in {1,2,4,8} */
  int32_t n_kv_heads; /* key/value heads                                                               */
  int32_t head_dim;   /* 64 or 128                                                                     */
  int32_t budget;     /* m of Algorithm 1: entries kept per lane after a step; 1 <= m < 2^20           */
  int32_t window;     /* W >= 1: the W newest entries are never picked (W = 1 is Algorithm 1's range
                         {0..m-1}; the Experiments section keeps 508 / 124 recent tokens)              */
  int32_t sink;       /* S >= 0: the S first tokens are never picked (Experiments section keeps 4);
                         budget >= sink + window is required                                           */
  int32_t dtype;      /* wkv_dtype: storage type of q, k, v, out and the cache                         */
  float scale;        /* softmax scale; 0 selects 1/sqrt(head_dim) (Ideal Merging section)             */
  int32_t merge;      /* 1: WeightedKV; 0: the "Eviction" variant of the Ablation Study (value dropped) */
  int32_t n_splits;   /* units a lane's cache scan is cut into; 0 = choose from the shape; max 64         */
  int32_t schedule;   /* wkv_schedule: how units are mapped to CTAs; 0 = choose from the shape            */
  void* stream;       /* cudaStream_t of the caller; NULL = the legacy default stream                  */
  wkv_alloc_fn alloc; /* NULL = cudaMalloc / cudaFree                                                  */
  wkv_release_fn release;
  void* user;
} wkv_config;

/* Host-only check of a configuration: NULL if wkv_create would accept it, else a static text naming the
 * first violated rule.  Touches no GPU. */
const char* wkv_config_error(const wkv_config* cfg);

/* Validates cfg, allocates the cache and bookkeeping for n_layers*batch*n_kv_heads lanes on the current
 * CUDA device through the provider and clears them (Algorithm 1 starts from empty score and count lists).  *out is
 * NULL on failure; when the provider returns NULL for one of the blocks the call returns WKV_ERR_ALLOC after handing
 * every block it had obtained back to `release`.  On bf16 rows the cache scan with four query heads per key, the value sweep of a blocked prompt tail and the
 * dense prompt kernel take tiles of the cache through tensor maps, which the driver encodes here (cuTensorMapEncodeTiled, looked up at run time): WKV_ERR_CUDA if
 * the driver lacks it, WKV_ERR_INVALID if the value cache would have 2^31 rows or more. */
int wkv_create(const wkv_config* cfg, wkv_ctx** out);

/* Releases everything obtained from the provider.  NULL is accepted. */
void wkv_destroy(wkv_ctx* ctx);

/* Empties every lane (all caches, scores, positions); asynchronous on the stream. */
int wkv_reset(wkv_ctx* ctx);

/* Changes the stream later calls are issued on.  The caller orders work across streams. */
int wkv_set_stream(wkv_ctx* ctx, void* stream);

/* One iteration of Algorithm 1 for every sequence of one layer (one or two kernel launches), asynchronous.
 *   q    device [batch, n_q_heads, head_dim]   query of the new token
 *   k, v device [batch, n_kv_heads, head_dim]  its key and value, appended to the cache first
 *                                              (Background: K_t = [K_{t-1}, k_t], V_t = [V_{t-1}, v_t])
 *   out  device [batch, n_q_heads, head_dim]   o_t = A_t^T V_t over the cache including the new token and
 *                                              before this step's merge
 *   evicted_pos device [batch, n_kv_heads] int32, or NULL: original 0-based position of the token whose
 *                                              key was dropped this step, -1 when the lane did not compress
 *   probs device [batch, n_q_heads, budget+1] fp32, or NULL: A_t in slot order (slot -> position through
 *                                              wkv_export_slots); slots beyond the lane's length get 0
 * Errors: WKV_ERR_INVALID (NULL ctx/q/k/v/out, layer out of range), WKV_ERR_CUDA (launch failure). */
int wkv_decode_step(wkv_ctx* ctx, int32_t layer, const void* q, const void* k, const void* v, void* out,
                    int32_t* evicted_pos, float* probs);

/* All layers of one decode step in one call: wkv_decode_step for layer 0, 1, ..., n_layers-1 (Algorithm 1 per lane;
 * the lanes of different layers are independent).
 *   q   device [n_layers, batch, n_q_heads, head_dim];  k, v device [n_layers, batch, n_kv_heads, head_dim]
 *   out device [n_layers, batch, n_q_heads, head_dim];  evicted_pos device [n_layers, batch, n_kv_heads] or NULL
 * By making this call the caller states that ALL layers' q, k, v are complete on the stream before it; the library
 * uses that to run the lanes of all layers in one launch when a layer alone is small, or else to let each layer's
 * cache scan run while the previous layer's per-lane epilogue is still finishing (results are identical to n_layers
 * separate calls).  Inputs must not overlap the outputs.  Asynchronous. */
int wkv_decode_step_layers(wkv_ctx* ctx, const void* q, const void* k, const void* v, void* out, int32_t* evicted_pos);

/* No counterpart in the paper: this entry point exists for callers that must not allocate device memory.
 *
 * Some hosts of this library cannot call cudaMalloc at the moment they need a decode step: code running
 * inside a region where allocation is forbidden or would stall (a latency-critical serving loop that
 * promised its allocator a fixed footprint, a process whose memory pool has been handed over entirely to
 * another component, a plug-in that is only allowed to use buffers it is given).  wkv_decode_step already
 * allocates nothing per call, but its scratch (parked logits, per-split partial outputs) was obtained from
 * the memory provider at wkv_create.  This variant runs the same two kernels (scan, lane epilogue) with that
 * scratch placed in a fixed array of WKV_STATIC_SCRATCH_BYTES bytes that is part of the library image, so a
 * context created through a provider that only hands out caller-owned memory never causes an allocation.
 * Every GPU that loads the library holds the array until the process exits.
 *
 *   Arguments, shapes and results: exactly those of wkv_decode_step, without `probs`.
 *   Limit: batch*n_kv_heads*(group*4*roundup4(budget+1) + n_splits*group*(head_dim+2)*4) bytes (each
 *          region rounded up to 256) must fit WKV_STATIC_SCRATCH_BYTES; otherwise WKV_ERR_INVALID is returned,
 *          nothing is launched, and wkv_last_error() names both numbers.
 *   First call on a device: looks up the array's device address (cudaGetSymbolAddress) with that device
 *          current and remembers it.  Make that first call outside any stream capture.
 *   Sharing: all contexts and all calls use the one array, which keeps the previous call's contents.  Nothing
 *          in it has to start at zero: every word the second kernel reads has been written by the first
 *          kernel of the same call.  Calls that can overlap on the GPU (different streams, or different contexts
 *          without ordering between them) race on the array: serialise them.
 *   Calls no cudaMalloc, cudaFree or other allocating routine.  (The CUDA runtime may load a kernel's code the
 *          first time that kernel is launched on a device and take device memory for it: run one step of the same
 *          shape outside the region that must not allocate.) */
#define WKV_STATIC_SCRATCH_BYTES (4u << 20)
int wkv_decode_step_static(wkv_ctx* ctx, int32_t layer, const void* q, const void* k, const void* v, void* out,
                           int32_t* evicted_pos);

/* The same step from HOST buffers: copies q, k, v to library-owned device staging, runs the step, copies
 * out (and evicted_pos if not NULL) back and waits for the stream.  Shapes as in wkv_decode_step. */
int wkv_decode_step_host(wkv_ctx* ctx, int32_t layer, const void* q, const void* k, const void* v, void* out,
                         int32_t* evicted_pos);

/* wkv_decode_step_layers from HOST buffers (shapes as there, all layers of one step): three copies in, the step, two
 * copies out, then waits for the stream. */
int wkv_decode_step_layers_host(wkv_ctx* ctx, const void* q, const void* k, const void* v, void* out,
                                int32_t* evicted_pos);

/* Consumes a prompt exactly as Algorithm 1 does: token by token, compressing as soon as a lane exceeds
 * the budget (the algorithm has no separate prompt phase).  One kernel launch per token, asynchronous.
 *   Q    device [batch, T_max, n_q_heads, head_dim], K, V device [batch, T_max, n_kv_heads, head_dim]
 *   seq_lens device [batch] int32 or NULL: sequence b consumes tokens 0..seq_lens[b]-1 (NULL = T_max each)
 *   out  device [batch, T_max, n_q_heads, head_dim] or NULL (outputs discarded into internal staging)
 *   evicted_pos device [batch, T_max, n_kv_heads] int32 or NULL */
int wkv_prefill(wkv_ctx* ctx, int32_t layer, const void* Q, const void* K, const void* V, const int32_t* seq_lens,
                int32_t T_max, void* out, int32_t* evicted_pos);

/* The same prompt, same arguments and same results as wkv_prefill, with the uncompressed part of the prompt done as
 * one dense problem per lane and the rest in blocks of tokens that share two sweeps of the cache.  Algorithm 1 compresses only once a lane holds more than `budget` entries; until then
 * its iterations are causal attention (Background section) plus the running sums of the attention columns.  The
 * library keeps, per layer, an upper bound on the tokens any lane has consumed since wkv_create / wkv_reset (calls of
 * every kind count; an imported lane counts as its token count if nothing of it was removed, as full otherwise).
 * While that bound is below the budget, the first min(T_max, budget - bound) tokens of the call go through one kernel
 * for all lanes of the layer -- on top of what each lane already holds, whose keys and values it reads from the cache
 * -- with every logit, probability and accumulated score computed by the arithmetic of the streamed step and the
 * scores added in the order of the tokens.  The remaining tokens are taken 8 / group at a time where window > 8 / group
 * and a lane's entries fit the register form of the per-lane kernel (budget + 1 <= 4352 for one query head per key):
 * one sweep over the key rows gives the logits of the whole block, the per-token step of Algorithm 1 (probabilities,
 * score fold, pick, merge) then runs on them token after token exactly as when streaming, and one sweep over the value
 * rows gives all outputs; elsewhere they are streamed as in wkv_prefill.  So a prompt may come in one call or in chunks.  K, positions, accumulated scores and removed positions are bit-identical to
 * wkv_prefill's; outputs and merged values agree within rounding.
 * The first call takes 64 * lanes_per_layer * round_up(budget, 128) bytes of scratch from the memory provider (twice that for
 * bf16 layers of at most two lanes per SM, which run blocks of 32 query rows), the first
 * blocked tail about 64 * lanes_per_layer * (budget + 1) bytes more (if the provider refuses those, the tail is streamed);
 * both are kept until wkv_destroy.  Q, K, V, out must be 16-byte aligned (WKV_ERR_INVALID otherwise).  Asynchronous. */
int wkv_prefill_bulk(wkv_ctx* ctx, int32_t layer, const void* Q, const void* K, const void* V, const int32_t* seq_lens,
                     int32_t T_max, void* out, int32_t* evicted_pos);

/* wkv_prefill_bulk for all layers of a prompt in one call (Algorithm 1 per lane; lanes of different layers are as
 * independent as lanes of one layer).
 *   Q device [n_layers, batch, T_max, n_q_heads, head_dim], K, V device [n_layers, batch, T_max, n_kv_heads, head_dim]
 *   seq_lens device [batch] or NULL (shared by the layers); out like Q or NULL; evicted_pos device
 *   [n_layers, batch, T_max, n_kv_heads] int32 or NULL.  Inputs and outputs must not overlap; 16-byte alignment as above.
 * While no lane of any layer can have reached the budget, the dense phase runs over the lanes of all layers at once if its scratch
 * (64 * n_layers * lanes_per_layer * round_up(budget, 128) bytes) stays under 256 MB -- what a single sequence needs to
 * fill the GPU -- and layer by layer otherwise.  The remaining tokens are streamed: one launch per token over the
 * lanes of all layers where wkv_decode_step_layers does the same, else with the layers interleaved so that one layer's
 * scan can run alongside the previous layer's lane epilogues.  Results equal wkv_prefill's. */
int wkv_prefill_bulk_layers(wkv_ctx* ctx, const void* Q, const void* K, const void* V, const int32_t* seq_lens,
                            int32_t T_max, void* out, int32_t* evicted_pos);

/* Copies one lane to HOST memory in position order and checks its bookkeeping (links form one chain of
 * `len` entries with strictly increasing positions); waits for the stream.  Any destination may be NULL.
 *   len, tokens : entries held / tokens consumed so far
 *   pos [len] int32 original positions; a [len] fp32 accumulated scores (n_i = tokens - pos_i);
 *   K, V [len, head_dim] storage type.  Buffers must have room for budget entries.
 * Returns WKV_ERR_STATE if the bookkeeping is inconsistent. */
int wkv_export_state(wkv_ctx* ctx, int32_t layer, int32_t b, int32_t kv_head, int32_t* len, int32_t* tokens,
                     int32_t* pos, float* a, void* K, void* V);

/* Slot-order view of one lane for interpreting `probs`: slot_pos [budget+1] int32 on the HOST, -1 for a
 * free slot.  Waits for the stream. */
int wkv_export_slots(wkv_ctx* ctx, int32_t layer, int32_t b, int32_t kv_head, int32_t* slot_pos);

/* Replaces one lane by the given position-ordered HOST state (len <= budget, pos strictly increasing and
 * < tokens).  Waits for the stream. */
int wkv_import_state(wkv_ctx* ctx, int32_t layer, int32_t b, int32_t kv_head, int32_t len, int32_t tokens,
                     const int32_t* pos, const float* a, const void* K, const void* V);

/* Reads and clears the device status word (waits for the stream): WKV_OK, WKV_ERR_TIMEOUT if a bounded wait inside
 * a kernel gave up since the last call, or WKV_ERR_STATE if a kernel found inconsistent slot links.
 * After WKV_ERR_TIMEOUT the context accepts calls as before (this call also clears the per-lane arrival counters of
 * the kernels), but a lane whose step was abandoned has consumed one token less than the others and its outputs of
 * that step are undefined: wkv_reset the context or wkv_import_state the affected lanes before decoding on. */
int wkv_status(wkv_ctx* ctx);

/* Self-test of the error path for device-side waits.  Every wait inside the kernels is bounded: the waits on a
 * shared-memory barrier fed by a bulk copy, and the lane epilogue's poll of its lane's arrival counter, which the scan
 * kernel in front of it increments (that kernel's CTAs have all started before an epilogue CTA becomes resident, so
 * the poll never waits for work that waits for it; at most 2^22 polls of about 100 ns).  After its limit the waiting
 * thread sets a bit in the device status word and carries on, so a kernel always terminates.  This call launches a
 * one-thread kernel that waits on a barrier nothing will complete (20000 polls, a few milliseconds); afterwards
 * wkv_status returns WKV_ERR_TIMEOUT once and the context is as usable as before.  Nothing faults or hangs.
 * Asynchronous. */
int wkv_selftest_wait_timeout(wkv_ctx* ctx);

/* Number of kernels this context has launched so far, and bytes it obtained from the provider. */
int64_t wkv_launch_count(const wkv_ctx* ctx);
int64_t wkv_device_bytes(const wkv_ctx* ctx);
/* The number of CTAs per lane the context uses (after resolving n_splits = 0); under the flat deal, where runs of tiles
 * cross lane boundaries, the largest number of CTAs that can share one lane. */
int32_t wkv_splits(const wkv_ctx* ctx);

const char* wkv_strerror(int code);
const char* wkv_last_error(const wkv_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* WKV_H_ */
