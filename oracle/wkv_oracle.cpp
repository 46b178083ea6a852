// WeightedKV reference oracle -- TEST INFRASTRUCTURE, not a product path.
//
// A plain, slow, list-based CPU restatement of the paper's Algorithm 1 (WeightedKV) and of the
// single-query attention of the Background section.  It exists to check the CUDA library and to be
// timed as a CPU baseline.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may
// load it.  It shares no code, header, table or constant generator with the CUDA library.
//
// One "lane" is one (layer, batch, kv-head): the paper drops the batch and head dimensions because
// every such lane runs the algorithm independently (Background, first paragraph).  Per lane the state
// is the paper's lists, kept in position order and physically erased on removal:
//   K, V  -- the key / value cache (Background: K_t = [K_{t-1}, k_t], V_t = [V_{t-1}, v_t]);
//   a     -- accumulated attention received by each retained token (Algorithm 1: a = [a,0] + A_t);
//   n     -- number of steps each retained token has been attended (Algorithm 1: n = [n,0] + 1).
//
// Two arithmetic modes:
//   mode 0 "double": every quantity in fp64.  This is the definition.
//   mode 1 "pinned": the chain that decides the eviction index (logits -> probabilities -> a -> a/n ->
//          argmin) and the merge weights are taken in a fully specified IEEE binary32 arithmetic (rules
//          P1..P7 below), so that an independent implementation can reproduce the eviction sequence
//          bit for bit.  The attention output o_t is still the fp64 definition in this mode.
//
// Readings of the paper taken here (the paper is silent or ambiguous on each):
//   * one loop iteration per incoming token (the loop variable of Algorithm 1 is garbled);
//   * logits are scaled by `scale`, default 1/sqrt(head_dim) (Ideal Merging section writes /sqrt(d));
//   * compression triggers when the list length EXCEEDS m (Algorithm 1; the worked example with
//     capacity 4 first compresses at step 5), so attention spans up to m+1 rows;
//   * the argmin runs over list indices [sink, L-1-window] (Algorithm 1 has sink=0, window=1: the newest
//     entry is never picked; the Experiments section keeps 4 initial and 508/124 recent tokens);
//   * ties go to the lowest position;
//   * the merge goes into the RIGHT neighbour, whose key, a and n are left untouched;
//   * the attention output uses V before the merge of the same step;
//   * the new token attends to itself and its own probability starts its a;
//   * if both average scores are zero the merge weights are (1/2, 1/2);
//   * grouped queries (G query heads per lane): a += mean over the group of the probabilities;
//   * storage type T (fp32 or bf16): inputs are T values; a merged value row is rounded to T
//     (round-to-nearest-even) when stored.
//
// Pinned binary32 rules (mode 1); every operation is IEEE-754 binary32 round-to-nearest-even,
// no flush-to-zero, no contraction except where fma is written:
//   P1 dot : 16 partial sums; partial r covers channels [r*d/16, (r+1)*d/16): its even channels and its odd
//            channels are each accumulated left to right as acc = fma(q_c, k_c, acc) from +0 and the two
//            chains are added.  Then four butterfly rounds p_r <- p_r + p_{r xor off}, off = 8,4,2,1.
//            s = scale32 * p_0, scale32 = (float) scale.
//   P2 max : M = max_i s_i;  x_i = s_i - M.
//   P3 exp : e = 0 if x < -87; else n = rint(x*LOG2E); f = fma(n,-LN2_HI,x); f = fma(n,-LN2_LO,f);
//            degree-7 Horner in fma with c_k = (float)(1/k!); e = poly * 2^n (exact).
//   P4 sum : E_i = trunc(e_i * 2^40) as a 64-bit integer; Z = (float)(sum_i E_i) * 2^-40.
//   P5 prob: p_i = e_i / Z.  Group mean: (((p0+p1)+p2)+...) * (float)(1/G), left to right.
//   P6 fold: a_i <- a_i + pbar_i;  abar_i = a_i / (float) n_i;  pick = lexicographic min of (abar, pos).
//   P7 merge: D = abar_j + abar_r; w_j = abar_j / D; w_r = abar_r / D;
//            v_c = fma(w_j, v_{j,c}, w_r * v_{r,c}); rounded to T.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

// ---- storage rounding ---------------------------------------------------------------------------
float bits_to_float(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }
uint32_t float_to_bits(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }

// binary32 -> bfloat16 (upper 16 bits of binary32), round to nearest, ties to even.
float round_float_to_bf16(float f) {
  if (std::isnan(f) || std::isinf(f)) return f;
  uint32_t u = float_to_bits(f);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  u &= 0xffff0000u;
  return bits_to_float(u);
}

// fp64 -> bfloat16 in one rounding (8 significant bits), ties to even (default rounding mode).
float round_double_to_bf16(double x) {
  if (x == 0.0 || std::isnan(x) || std::isinf(x)) return (float)x;
  int e;
  std::frexp(x, &e);                       // x = m * 2^e, 0.5 <= |m| < 1
  int q = e - 8;                           // quantum exponent for 8 significant bits
  if (q < -133) q = -133;                  // subnormal range of the binary32 exponent field
  double y = std::nearbyint(std::ldexp(x, -q));
  return (float)std::ldexp(y, q);
}

enum { T_F32 = 0, T_BF16 = 1 };

float store_from_double(double x, int dtype) { return dtype == T_BF16 ? round_double_to_bf16(x) : (float)x; }
float store_from_float(float x, int dtype) { return dtype == T_BF16 ? round_float_to_bf16(x) : x; }

// ---- pinned binary32 pieces -----------------------------------------------------------------------
// P1
float pinned_dot(const float* q, const float* k, int d, float scale32) {
  float p[16];
  const int w = d / 16;
  for (int r = 0; r < 16; ++r) {
    float even = 0.0f, odd = 0.0f;
    for (int c = r * w; c < (r + 1) * w; ++c) {
      if ((c - r * w) % 2 == 0) even = std::fmaf(q[c], k[c], even);
      else odd = std::fmaf(q[c], k[c], odd);
    }
    p[r] = even + odd;
  }
  for (int off = 8; off >= 1; off >>= 1) {
    float nxt[16];
    for (int r = 0; r < 16; ++r) nxt[r] = p[r] + p[r ^ off];
    for (int r = 0; r < 16; ++r) p[r] = nxt[r];
  }
  return scale32 * p[0];
}

// P3
float pinned_exp(float x) {
  const float LOG2E  = bits_to_float(0x3fb8aa3bu);   // (float) log2(e)
  const float LN2_HI = bits_to_float(0x3f317000u);   // (float) ln 2 with the low 12 significand bits cleared
  const float LN2_LO = bits_to_float(0x3805fdf4u);   // (float)(ln 2 - LN2_HI)
  if (x < -87.0f) return 0.0f;
  float n = std::rint(x * LOG2E);
  float f = std::fmaf(n, -LN2_HI, x);
  f = std::fmaf(n, -LN2_LO, f);
  const float c2 = 0.5f, c3 = (float)(1.0 / 6.0), c4 = (float)(1.0 / 24.0), c5 = (float)(1.0 / 120.0),
              c6 = (float)(1.0 / 720.0), c7 = (float)(1.0 / 5040.0);
  float r = c7;
  r = std::fmaf(r, f, c6);
  r = std::fmaf(r, f, c5);
  r = std::fmaf(r, f, c4);
  r = std::fmaf(r, f, c3);
  r = std::fmaf(r, f, c2);
  r = std::fmaf(r, f, 1.0f);
  r = std::fmaf(r, f, 1.0f);
  return std::ldexp(r, (int)n);            // exact: the result stays a normal binary32 number
}

// P2..P5 for one query head: logits s[0..L) -> probabilities p[0..L)
void pinned_softmax(const std::vector<float>& s, std::vector<float>& p) {
  const size_t L = s.size();
  float M = s[0];
  for (size_t i = 1; i < L; ++i) M = std::max(M, s[i]);
  std::vector<float> e(L);
  uint64_t zint = 0;
  for (size_t i = 0; i < L; ++i) {
    e[i] = pinned_exp(s[i] - M);
    zint += (uint64_t)(e[i] * 1099511627776.0f);     // trunc(e * 2^40); the product is exact
  }
  const float Z = (float)zint * (1.0f / 1099511627776.0f);
  p.resize(L);
  for (size_t i = 0; i < L; ++i) p[i] = e[i] / Z;
}

struct Lane {
  std::vector<std::vector<float>> K, V;    // list order == position order; entries are T values
  std::vector<double> a_d;                 // mode 0
  std::vector<float> a_f;                  // mode 1
  std::vector<int64_t> n;                  // Algorithm 1's count list
  std::vector<int32_t> pos;                // original (0-based) position of the token whose key the entry holds
  std::vector<int32_t> cnt;                // how many original tokens are mixed into V[i]
  std::vector<std::vector<double>> C;      // optional: mixture coefficients of V[i] over original tokens
  int64_t t = 0;                           // tokens consumed so far
  double dropped_a = 0.0;                  // sum of a over removed entries (bookkeeping invariant)
  // record of the last step
  int32_t last_evicted_pos = -1;
  int32_t last_evicted_index = -1;
  double last_wj = 0.0, last_wr = 0.0;
  double last_prob_sum = 0.0;
  // the pick of the last compressing step: what the lane's own argmin chose and what was removed (they differ only
  // when the caller imposed the removal, see wkvo_impose_pick)
  int32_t last_own_pos = -1;
  double last_own_abar = 0.0, last_taken_abar = 0.0;
  int32_t imposed_pos = -1;                // one-shot: position to remove at the next compressing step, -1 = own argmin
  int32_t last_imposed_bad = 0;            // the imposed position was not in the evictable range (own argmin used)
};

}  // namespace

extern "C" {

typedef struct {
  int32_t n_lanes;     // independent lanes
  int32_t group;       // G: query heads per lane (1 = multi-head attention)
  int32_t head_dim;    // d, a multiple of 16
  int32_t budget;      // m  (Algorithm 1 input)
  int32_t window;      // most recent entries never picked (>= 1)
  int32_t sink;        // initial tokens never picked (>= 0)
  int32_t dtype;       // 0 = fp32 storage, 1 = bf16 storage
  int32_t mode;        // 0 = double, 1 = pinned
  int32_t merge;       // 1 = WeightedKV; 0 = the "Eviction" ablation (Ablation Study): value dropped too
  int32_t track;       // 1 = track mixture coefficients (tiny inputs only)
  double scale;        // softmax scale; 0 -> 1/sqrt(head_dim)
} wkvo_config;

struct wkvo {
  wkvo_config cfg;
  double scale;
  float scale32;
  std::vector<Lane> lanes;
};

wkvo* wkvo_create(const wkvo_config* c) {
  if (!c || c->n_lanes < 1 || c->group < 1 || c->head_dim < 16 || c->head_dim % 16 || c->budget < 1 ||
      c->window < 1 || c->sink < 0 || c->budget < c->sink + c->window)
    return nullptr;
  wkvo* o = new wkvo;
  o->cfg = *c;
  o->scale = c->scale != 0.0 ? c->scale : 1.0 / std::sqrt((double)c->head_dim);
  o->scale32 = (float)o->scale;
  o->lanes.resize(c->n_lanes);
  return o;
}

void wkvo_destroy(wkvo* o) { delete o; }

// One token for every active lane (Algorithm 1, one loop iteration per lane).
//   q [n_lanes, G, d], k, v [n_lanes, d] : fp32 arrays holding T values (rounded to T here regardless)
//   active [n_lanes] or NULL            : lanes with 0 are left untouched (ragged batches)
//   out [n_lanes, G, d] or NULL         : attention output o_t, unrounded fp64
//   evicted [n_lanes] or NULL           : original position of the removed key, -1 if none
//   probs [n_lanes, G, budget+1] or NULL: A_t in list order (fp64; the pinned values in mode 1)
void wkvo_step(wkvo* o, const float* q, const float* k, const float* v, const uint8_t* active, double* out,
               int32_t* evicted, double* probs) {
  const wkvo_config& c = o->cfg;
  const int d = c.head_dim, G = c.group, m = c.budget;
#pragma omp parallel for schedule(dynamic, 1)
  for (int ln = 0; ln < c.n_lanes; ++ln) {
    if (active && !active[ln]) {
      if (evicted) evicted[ln] = -1;
      continue;
    }
    Lane& S = o->lanes[ln];
    const int64_t t = S.t;
    // Background: K_t = [K_{t-1}, k_t], V_t = [V_{t-1}, v_t];  Algorithm 1: [a,0], [n,0].
    std::vector<float> kr(d), vr(d);
    for (int ch = 0; ch < d; ++ch) {
      kr[ch] = store_from_float(k[(size_t)ln * d + ch], c.dtype);
      vr[ch] = store_from_float(v[(size_t)ln * d + ch], c.dtype);
    }
    S.K.push_back(kr);
    S.V.push_back(vr);
    S.a_d.push_back(0.0);
    S.a_f.push_back(0.0f);
    S.n.push_back(0);
    S.pos.push_back((int32_t)t);
    S.cnt.push_back(1);
    if (c.track) {
      for (auto& row : S.C) row.push_back(0.0);
      std::vector<double> row((size_t)t + 1, 0.0);
      row[(size_t)t] = 1.0;
      S.C.push_back(row);
    }
    const int L = (int)S.K.size();

    // In mode 1 the fp64 probabilities serve the output only: a caller that asks for no output does not pay for them.
    const bool need_fp64 = c.mode == 0 || out != nullptr;
    std::vector<std::vector<double>> pd(G, std::vector<double>(need_fp64 ? L : 0));
    std::vector<std::vector<float>> pf(G);
    for (int g = 0; g < G; ++g) {
      std::vector<float> qr(d);
      for (int ch = 0; ch < d; ++ch) qr[ch] = store_from_float(q[((size_t)ln * G + g) * d + ch], c.dtype);
      if (need_fp64) {
        // Background: A_t = softmax(q_t^T K_t) (scaled), o_t = A_t^T V_t -- the fp64 definition.
        std::vector<double> s(L);
        double M = -INFINITY;
        for (int i = 0; i < L; ++i) {
          double acc = 0.0;
          for (int ch = 0; ch < d; ++ch) acc += (double)qr[ch] * (double)S.K[i][ch];
          s[i] = o->scale * acc;
          M = std::max(M, s[i]);
        }
        double Z = 0.0;
        for (int i = 0; i < L; ++i) { pd[g][i] = std::exp(s[i] - M); Z += pd[g][i]; }
        for (int i = 0; i < L; ++i) pd[g][i] /= Z;
      }
      if (out) {
        for (int ch = 0; ch < d; ++ch) {
          double acc = 0.0;
          for (int i = 0; i < L; ++i) acc += pd[g][i] * (double)S.V[i][ch];   // V before this step's merge
          out[((size_t)ln * G + g) * d + ch] = acc;
        }
      }
      if (c.mode == 1) {
        std::vector<float> sf(L);
        for (int i = 0; i < L; ++i) sf[i] = pinned_dot(qr.data(), S.K[i].data(), d, o->scale32);
        pinned_softmax(sf, pf[g]);
      }
      if (probs) {
        double* dst = probs + ((size_t)ln * G + g) * (size_t)(m + 1);
        for (int i = 0; i < m + 1; ++i) dst[i] = i < L ? (c.mode == 1 ? (double)pf[g][i] : pd[g][i]) : 0.0;
      }
    }

    // Algorithm 1: a = [a,0] + A_t ; n = [n,0] + 1   (group mean of A_t over the G query heads)
    double psum = 0.0;
    for (int i = 0; i < L; ++i) {
      if (c.mode == 1) {
        float acc = pf[0][i];
        for (int g = 1; g < G; ++g) acc = acc + pf[g][i];
        if (G > 1) acc = acc * (float)(1.0 / (double)G);
        S.a_f[i] = S.a_f[i] + acc;
        psum += (double)acc;
      } else {
        double acc = 0.0;
        for (int g = 0; g < G; ++g) acc += pd[g][i];
        acc /= (double)G;
        S.a_d[i] += acc;
        psum += acc;
      }
      S.n[i] += 1;
    }
    S.last_prob_sum = psum;
    S.last_evicted_pos = -1;
    S.last_evicted_index = -1;
    S.last_wj = S.last_wr = 0.0;

    // Algorithm 1: if the length of V_t exceeds m
    if (L > m) {
      // abar = a / n ;  j = argmin over the evictable range, first minimiser (lowest position)
      const int lo = c.sink, hi = L - 1 - c.window;    // inclusive list-index range
      int j = -1;
      if (c.mode == 1) {
        float best = 0.0f;
        for (int i = lo; i <= hi; ++i) {
          float ab = S.a_f[i] / (float)S.n[i];
          if (j < 0 || ab < best) { best = ab; j = i; }
        }
      } else {
        double best = 0.0;
        for (int i = lo; i <= hi; ++i) {
          double ab = S.a_d[i] / (double)S.n[i];
          if (j < 0 || ab < best) { best = ab; j = i; }
        }
      }
      // (budget >= sink + window guarantees lo <= hi, so j >= 0 and j+1 exists)
      auto abar_of = [&](int i) {
        return c.mode == 1 ? (double)(S.a_f[i] / (float)S.n[i]) : S.a_d[i] / (double)S.n[i];
      };
      S.last_own_pos = S.pos[j];
      S.last_own_abar = abar_of(j);
      S.last_imposed_bad = 0;
      if (S.imposed_pos >= 0) {
        // A caller-imposed removal (wkvo_impose_pick) replaces the lane's own argmin for this one step.
        int forced = -1;
        for (int i = lo; i <= hi; ++i)
          if (S.pos[i] == S.imposed_pos) forced = i;
        if (forced >= 0) j = forced; else S.last_imposed_bad = 1;
        S.imposed_pos = -1;
      }
      S.last_taken_abar = abar_of(j);
      const int r = j + 1;
      double wj, wr;
      if (c.mode == 1) {
        const float aj = S.a_f[j] / (float)S.n[j], ar = S.a_f[r] / (float)S.n[r];
        const float D = aj + ar;
        float fwj, fwr;
        if (D == 0.0f) { fwj = 0.5f; fwr = 0.5f; } else { fwj = aj / D; fwr = ar / D; }
        if (c.merge)
          for (int ch = 0; ch < d; ++ch)
            S.V[r][ch] = store_from_float(std::fmaf(fwj, S.V[j][ch], fwr * S.V[r][ch]), c.dtype);
        wj = fwj; wr = fwr;
      } else {
        const double aj = S.a_d[j] / (double)S.n[j], ar = S.a_d[r] / (double)S.n[r];
        const double D = aj + ar;
        if (D == 0.0) { wj = 0.5; wr = 0.5; } else { wj = aj / D; wr = ar / D; }
        // Algorithm 1: V[j:j+2] <- (abar_j V_j + abar_{j+1} V_{j+1}) / (abar_j + abar_{j+1})
        if (c.merge)
          for (int ch = 0; ch < d; ++ch)
            S.V[r][ch] = store_from_double(wj * (double)S.V[j][ch] + wr * (double)S.V[r][ch], c.dtype);
      }
      if (c.merge) {
        S.cnt[r] += S.cnt[j];
        if (c.track)
          for (size_t u = 0; u < S.C[r].size(); ++u) S.C[r][u] = wj * S.C[j][u] + wr * S.C[r][u];
      }
      S.last_evicted_pos = S.pos[j];
      S.last_evicted_index = j;
      S.last_wj = wj;
      S.last_wr = wr;
      S.dropped_a += c.mode == 1 ? (double)S.a_f[j] : S.a_d[j];
      // Algorithm 1: remove K[j], a[j], n[j] (the merged pair now occupies one entry)
      S.K.erase(S.K.begin() + j);
      S.V.erase(S.V.begin() + j);
      S.a_d.erase(S.a_d.begin() + j);
      S.a_f.erase(S.a_f.begin() + j);
      S.n.erase(S.n.begin() + j);
      S.pos.erase(S.pos.begin() + j);
      S.cnt.erase(S.cnt.begin() + j);
      if (c.track) S.C.erase(S.C.begin() + j);
    }
    if (evicted) evicted[ln] = S.last_evicted_pos;
    S.t = t + 1;
  }
}

int32_t wkvo_len(const wkvo* o, int32_t lane) { return (int32_t)o->lanes[lane].K.size(); }
int64_t wkvo_tokens(const wkvo* o, int32_t lane) { return o->lanes[lane].t; }
double wkvo_dropped_score(const wkvo* o, int32_t lane) { return o->lanes[lane].dropped_a; }

// Record of the lane's most recent step: removed list index (-1 = none), merge weights, sum of folded probabilities.
void wkvo_last_step(const wkvo* o, int32_t lane, int32_t* index, double* wj, double* wr, double* prob_sum) {
  const Lane& S = o->lanes[lane];
  if (index) *index = S.last_evicted_index;
  if (wj) *wj = S.last_wj;
  if (wr) *wr = S.last_wr;
  if (prob_sum) *prob_sum = S.last_prob_sum;
}

// Test hook for comparing two arithmetic modes on one stream.  Algorithm 1 removes the argmin of the average scores;
// where the two smallest averages lie closer together than binary32 rounding noise, mode 0 and mode 1 may legitimately
// pick different entries, after which their states are no longer comparable.  wkvo_impose_pick makes every lane with
// pos[lane] >= 0 remove the entry at that original position on its NEXT compressing step instead of its own argmin
// (the position must lie in the evictable range, else the lane keeps its own choice and reports it); wkvo_last_pick
// then tells what the lane would have picked by itself and the average scores of both entries, so that the caller can
// check that the imposed entry was a near-minimum.  Everything else of the step is unchanged.
void wkvo_impose_pick(wkvo* o, const int32_t* pos) {
  for (int32_t ln = 0; ln < o->cfg.n_lanes; ++ln) o->lanes[ln].imposed_pos = pos ? pos[ln] : -1;
}
void wkvo_last_pick(const wkvo* o, int32_t lane, int32_t* own_pos, double* own_abar, double* taken_abar, int32_t* imposed_bad) {
  const Lane& S = o->lanes[lane];
  if (own_pos) *own_pos = S.last_own_pos;
  if (own_abar) *own_abar = S.last_own_abar;
  if (taken_abar) *taken_abar = S.last_taken_abar;
  if (imposed_bad) *imposed_bad = S.last_imposed_bad;
}

// Position-ordered copy of a lane.  Any destination may be NULL.
//   pos, cnt [len] int32; n [len] int64; a [len] fp64; K, V [len, d] fp32;
//   coeff [len, tokens] fp64 (only when created with track = 1)
void wkvo_export(const wkvo* o, int32_t lane, int32_t* pos, int64_t* n, double* a, float* K, float* V, int32_t* cnt,
                 double* coeff) {
  const Lane& S = o->lanes[lane];
  const int d = o->cfg.head_dim;
  const size_t L = S.K.size();
  for (size_t i = 0; i < L; ++i) {
    if (pos) pos[i] = S.pos[i];
    if (n) n[i] = S.n[i];
    if (a) a[i] = o->cfg.mode == 1 ? (double)S.a_f[i] : S.a_d[i];
    if (cnt) cnt[i] = S.cnt[i];
    if (K) std::memcpy(K + i * d, S.K[i].data(), sizeof(float) * d);
    if (V) std::memcpy(V + i * d, S.V[i].data(), sizeof(float) * d);
    if (coeff && o->cfg.track)
      for (size_t u = 0; u < (size_t)S.t; ++u) coeff[i * (size_t)S.t + u] = u < S.C[i].size() ? S.C[i][u] : 0.0;
  }
}

// Replaces a lane by the given position-ordered state (test set-up for large caches: filling them token by token
// would take the tests minutes).  tokens = tokens consumed so far; Algorithm 1's count of entry i is then
// tokens - pos[i].  Multiplicities restart at 1; not available with coefficient tracking.
int32_t wkvo_import(wkvo* o, int32_t lane, int32_t len, int64_t tokens, const int32_t* pos, const double* a, const float* K,
                    const float* V) {
  if (o->cfg.track || len < 0 || len > o->cfg.budget || tokens < len) return -1;
  Lane& S = o->lanes[lane];
  const int d = o->cfg.head_dim;
  S = Lane();
  S.t = tokens;
  for (int32_t i = 0; i < len; ++i) {
    if (pos[i] < 0 || pos[i] >= tokens || (i > 0 && pos[i] <= pos[i - 1])) return -1;
    S.K.emplace_back(K + (size_t)i * d, K + (size_t)(i + 1) * d);
    S.V.emplace_back(V + (size_t)i * d, V + (size_t)(i + 1) * d);
    S.a_d.push_back(a[i]);
    S.a_f.push_back((float)a[i]);
    S.n.push_back(tokens - pos[i]);
    S.pos.push_back(pos[i]);
    S.cnt.push_back(1);
  }
  return 0;
}

// The pinned pieces, exposed so the tests can pin them against libm / fp64.
float wkvo_pinned_exp(float x) { return pinned_exp(x); }
float wkvo_pinned_dot(const float* q, const float* k, int32_t d, float scale32) { return pinned_dot(q, k, d, scale32); }
void wkvo_pinned_softmax(const float* s, int32_t L, float* p) {
  std::vector<float> sv(s, s + L), pv;
  pinned_softmax(sv, pv);
  std::memcpy(p, pv.data(), sizeof(float) * L);
}
float wkvo_round_bf16(float x) { return round_float_to_bf16(x); }
float wkvo_round_bf16_from_double(double x) { return round_double_to_bf16(x); }

}  // extern "C"
