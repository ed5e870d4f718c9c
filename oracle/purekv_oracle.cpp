// CPU oracle for the PureKV hot path.  TEST INFRASTRUCTURE ONLY: slow, plain,
// fp64, written from the paper's definitions.  It shares no code with the CUDA
// library and must never be called from the product path; only the tests, the
// smoke check and the benchmark's CPU-baseline leg use it.
//
// What each function follows:
//   pko_mask           ST-SpAttn mask, Sec. 3.2 (spatial path: first frame + current
//                      frame; temporal path: corresponding token of the previous frame
//                      + first frame), under causal attention (Sec. 3.1/3.2); the comparison
//                      masks of App. A.3 / Table 7 (spatial only, temporal only, local,
//                      atrous) and a block-level widening of any of them.
//   pko_prefill        masked softmax attention; the softmax is Eq. 1 restricted to the
//                      kept keys of each row.
//   pko_lowlayer_score Eq. 1 (dense causal softmax rows) and Eq. 2 (sum of the recent
//                      window's rows over the non-recent keys).
//   pko_lowlayer_score_ex  the same with the other reductions of App. A.1 / Table 6's policies
//                      (accumulation over all rows, an observation window, pooling along keys).
//   pko_select_sink_recent  the score-free policy of App. A.1 / Table 6 (first keys + window).
//   pko_spearman       Eq. 7, the rank correlation of Sec. 3.3 (validation tool, CPU only).
//   pko_vnorm_scores   Eq. 3 / Eq. 4 (C weighted by the L2 norm of each key's V vector).
//   pko_select         Sec. 3.1: keep the recent window w plus the top-h non-recent keys.
//   pko_compact        the compacted cache implied by that selection.
//   pko_budget         integer budget from a keep ratio.
//   pko_decode         one decoding step over the compacted cache (the stage Table 3 times as
//                      decode latency): the new token's softmax attention, Eq. 1 for a single
//                      row, over the keys its request kept; every kept key is visible.
// Readings taken where the paper is silent: visual tokens in raster order inside a frame;
// prefix tokens visible to every query and text rows dense causal; the spatial and the
// temporal path form one mask (their union); softmax rows of Eq. 1 normalised over the
// whole causal row; C of a KV head is the mean over its group's query heads; V norms
// per KV head; the budget counts the recent window; ties in the top-h cut go to the
// lower position and the chosen positions are listed in ascending order.
//
// Parity pins: every function here is pinned by the CPU tests against brute
// force, closed forms, invariants or library special cases.  Nothing numeric is
// printed by the paper for these operations, so agreement with the authors' own
// (unpublished) implementation is "parity unpinned".
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>

extern "C" {

struct pko_mask_params {
  int32_t grid_h, grid_w;
  int32_t anchor_frames;    // first frames every visual query sees (paper: 1)
  int32_t spatial_radius;   // -1: whole current frame (paper); else Chebyshev radius
  int32_t temporal_depth;   // number of linked earlier frames (paper: 1), -1: all
  int32_t temporal_stride;  // linked frames are f-s, f-2s, ... (paper: 1)
  int32_t temporal_radius;  // 0: same grid cell only (paper); -1: whole linked frame
  int32_t dense_causal;     // nonzero: plain causal attention
  // The comparison masks of App. A.3 / Table 7 (the paper names them and shows them only in a figure that the text
  // does not reproduce; the readings are the usual meanings of the names):
  int32_t local_window;     // > 0: Local Attention -- a visual query also sees the local_window most recent positions
  int32_t atrous_dilation;  // > 0: Atrous Attention -- a visual query also sees every atrous_dilation-th earlier position
  int32_t coarse_block;     // > 0: the mask is widened to blocks of this many positions (a block pair is kept whole,
                            //      under causality, as soon as it holds one kept pair): block-sparse reading of the mask
};

// The token-level predicate.  Sec. 3.2 for the spatial and temporal paths; App. A.3 names the other two.
static int32_t mask_token(const pko_mask_params* p, int32_t len, int32_t n_prefix, int32_t n_frames, int32_t i,
                          int32_t j) {
  if (i < 0 || j < 0 || i >= len || j >= len) return 0;
  if (j > i) return 0;                           // causal attention
  if (p->dense_causal) return 1;
  const int32_t n = p->grid_h * p->grid_w;
  const int32_t vis_end = n_prefix + n_frames * n;
  const bool i_visual = i >= n_prefix && i < vis_end;
  if (!i_visual) return 1;                       // text queries: dense causal
  if (j < n_prefix) return 1;                    // prefix keys: always visible
  // both visual (j <= i < vis_end and j >= n_prefix)
  const int32_t fi = (i - n_prefix) / n, pi = (i - n_prefix) % n;
  const int32_t fj = (j - n_prefix) / n, pj = (j - n_prefix) % n;
  const int32_t yi = pi / p->grid_w, xi = pi % p->grid_w;
  const int32_t yj = pj / p->grid_w, xj = pj % p->grid_w;
  const int32_t rho = std::max(std::abs(yi - yj), std::abs(xi - xj));
  const int32_t df = fi - fj;
  // (1) attention to the first frame(s): both paths keep it
  if (fj < p->anchor_frames) return 1;
  // (2) spatial path: the current frame
  if (df == 0 && (p->spatial_radius < 0 || rho <= p->spatial_radius)) return 1;
  // (3) temporal path: the corresponding token of the previous frame(s)
  if (df >= 1 && p->temporal_stride >= 1 && df % p->temporal_stride == 0 &&
      (p->temporal_depth < 0 || df <= (int64_t)p->temporal_depth * p->temporal_stride) &&
      (p->temporal_radius < 0 || rho <= p->temporal_radius))
    return 1;
  // (4) Local Attention: the most recent positions, whatever frame they belong to
  if (p->local_window > 0 && i - j < p->local_window) return 1;
  // (5) Atrous Attention: every dilation-th position counted back from the query
  if (p->atrous_dilation > 0 && (i - j) % p->atrous_dilation == 0) return 1;
  return 0;
}

// Positions are relative to the request; len = n_prefix + n_frames*N + n_suffix.
// Returns 1 when query i may attend key j.
int32_t pko_mask(const pko_mask_params* p, int32_t len, int32_t n_prefix, int32_t n_frames,
                 int32_t i, int32_t j) {
  if (p->coarse_block <= 0 || p->dense_causal) return mask_token(p, len, n_prefix, n_frames, i, j);
  if (i < 0 || j < 0 || i >= len || j > i) return 0;
  // block-level reading: (i, j) is kept if its block pair holds any kept pair of the token-level mask
  const int32_t B = p->coarse_block, i0 = (i / B) * B, j0 = (j / B) * B;
  for (int32_t ii = i0; ii < std::min(len, i0 + B); ++ii)
    for (int32_t jj = j0; jj < std::min(len, j0 + B); ++jj)
      if (mask_token(p, len, n_prefix, n_frames, ii, jj)) return 1;
  return 0;
}

void pko_mask_matrix(const pko_mask_params* p, int32_t len, int32_t n_prefix, int32_t n_frames,
                     uint8_t* out /* [len*len] */) {
  for (int32_t i = 0; i < len; ++i)
    for (int32_t j = 0; j < len; ++j)
      out[(int64_t)i * len + j] = (uint8_t)pko_mask(p, len, n_prefix, n_frames, i, j);
}

static inline double dot_fd(const float* a, const float* b, int32_t d) {
  double s = 0.0;
  for (int32_t c = 0; c < d; ++c) s += (double)a[c] * (double)b[c];
  return s;
}

// Masked softmax attention for a list of rows and heads.
// q [T,H,d], k,v [T,H_kv,d] float32 (bf16 inputs are passed widened, which is exact).
// rows: absolute token indices (NULL = all T rows); heads: query heads (NULL = all).
// out [n_rows, n_heads, d] float64, lse [n_heads, n_rows] float64 (natural log).
// scale <= 0 means 1/sqrt(d) (Eq. 1).
void pko_prefill(const float* q, const float* k, const float* v,
                 int32_t n_req, const int32_t* cu_seqlens, const int32_t* n_prefix,
                 const int32_t* n_frames, const pko_mask_params* mp,
                 int32_t n_q_heads, int32_t n_kv_heads, int32_t d, double scale,
                 const int64_t* rows, int64_t n_rows, const int32_t* heads, int32_t n_heads,
                 double* out, double* lse) {
  const int64_t T = cu_seqlens[n_req];
  if (!rows) n_rows = T;
  if (!heads) n_heads = n_q_heads;
  if (scale <= 0.0) scale = 1.0 / std::sqrt((double)d);
  const int32_t G = n_q_heads / n_kv_heads;
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t ri = 0; ri < n_rows; ++ri) {
    const int64_t t = rows ? rows[ri] : ri;
    int32_t r = 0;
    while (r + 1 < n_req && t >= cu_seqlens[r + 1]) ++r;
    const int64_t base = cu_seqlens[r];
    const int32_t len = cu_seqlens[r + 1] - cu_seqlens[r];
    const int32_t i = (int32_t)(t - base);
    std::vector<double> s(i + 1);
    std::vector<uint8_t> keep(i + 1);
    for (int32_t j = 0; j <= i; ++j) keep[j] = (uint8_t)pko_mask(mp, len, n_prefix[r], n_frames[r], i, j);
    for (int32_t hi = 0; hi < n_heads; ++hi) {
      const int32_t hq = heads ? heads[hi] : hi;
      const int32_t g = hq / G;
      const float* qi = q + ((int64_t)t * n_q_heads + hq) * d;
      double m = -std::numeric_limits<double>::infinity();
      for (int32_t j = 0; j <= i; ++j) {
        if (!keep[j]) continue;
        s[j] = scale * dot_fd(qi, k + ((base + j) * n_kv_heads + g) * d, d);
        m = std::max(m, s[j]);
      }
      double z = 0.0;
      double* o = out + ((int64_t)ri * n_heads + hi) * d;
      for (int32_t c = 0; c < d; ++c) o[c] = 0.0;
      for (int32_t j = 0; j <= i; ++j) {
        if (!keep[j]) continue;
        const double e = std::exp(s[j] - m);
        z += e;
        const float* vj = v + ((base + j) * n_kv_heads + g) * d;
        for (int32_t c = 0; c < d; ++c) o[c] += e * (double)vj[c];
      }
      for (int32_t c = 0; c < d; ++c) o[c] /= z;
      if (lse) lse[(int64_t)hi * n_rows + ri] = m + std::log(z);
    }
  }
}

// Eq. 1 + Eq. 2.  For every request and KV head g:
//   C[g, j] = (1/G) sum_{hq in group g} sum_{i=l-w}^{l-1} A^{hq}_{i,j},  0 <= j < l-w,
// with A the dense causal softmax (row i normalised over all j' <= i).  The mean
// over the group's query heads is this build's reading (the paper is silent on GQA).
// c_out [H_kv, T] float64; entries of each request's last w positions are set to 0.
// The window is clipped to the request length.
void pko_lowlayer_score(const float* q, const float* k,
                        int32_t n_req, const int32_t* cu_seqlens, int32_t window,
                        int32_t n_q_heads, int32_t n_kv_heads, int32_t d, double scale,
                        double* c_out) {
  const int64_t T = cu_seqlens[n_req];
  if (scale <= 0.0) scale = 1.0 / std::sqrt((double)d);
  const int32_t G = n_q_heads / n_kv_heads;
  for (int64_t x = 0; x < (int64_t)n_kv_heads * T; ++x) c_out[x] = 0.0;
  for (int32_t r = 0; r < n_req; ++r) {
    const int64_t base = cu_seqlens[r];
    const int32_t len = cu_seqlens[r + 1] - cu_seqlens[r];
    const int32_t w = std::min(window, len);
    const int32_t nr = len - w;                       // non-recent keys: 0 .. nr-1
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t g = 0; g < n_kv_heads; ++g) {
      std::vector<double> s(len), acc(std::max(nr, 1), 0.0);
      for (int32_t hq = g * G; hq < (g + 1) * G; ++hq) {
        for (int32_t i = len - w; i < len; ++i) {
          const float* qi = q + ((base + i) * n_q_heads + hq) * d;
          double m = -std::numeric_limits<double>::infinity();
          for (int32_t j = 0; j <= i; ++j) {
            s[j] = scale * dot_fd(qi, k + ((base + j) * n_kv_heads + g) * d, d);
            m = std::max(m, s[j]);
          }
          double z = 0.0;
          for (int32_t j = 0; j <= i; ++j) { s[j] = std::exp(s[j] - m); z += s[j]; }
          for (int32_t j = 0; j < nr; ++j) acc[j] += s[j] / z;
        }
      }
      for (int32_t j = 0; j < nr; ++j) c_out[(int64_t)g * T + base + j] = acc[j] / (double)G;
    }
  }
}

// The score reductions of the policies the paper combines its estimator with (App. A.1, Table 6), as variations of
// Eq. 2 (the paper cites them by name; the forms below are the usual ones of those methods):
//   accumulated attention (Sec. 3.1: "most existing methods rely on accumulated attention scores", which the
//     lower-triangular matrix biases toward early tokens): every row of A is summed, obs_rows < 0 or >= l;
//   an observation window of obs_rows last rows (obs_rows = window is Eq. 2 itself);
//   pooling along the key axis: pool > 1 replaces each non-recent key's sum by the mean over the pool positions
//     centred on it, positions outside the non-recent segment counting as 0 (pool odd).
// A row contributes to the keys it can see (j <= i) only.  Rows, normalisation, GQA mean and output layout as in
// pko_lowlayer_score.
void pko_lowlayer_score_ex(const float* q, const float* k, int32_t n_req, const int32_t* cu_seqlens, int32_t window,
                           int32_t obs_rows, int32_t pool, int32_t n_q_heads, int32_t n_kv_heads, int32_t d,
                           double scale, double* c_out) {
  const int64_t T = cu_seqlens[n_req];
  if (scale <= 0.0) scale = 1.0 / std::sqrt((double)d);
  const int32_t G = n_q_heads / n_kv_heads;
  for (int64_t x = 0; x < (int64_t)n_kv_heads * T; ++x) c_out[x] = 0.0;
  for (int32_t r = 0; r < n_req; ++r) {
    const int64_t base = cu_seqlens[r];
    const int32_t len = cu_seqlens[r + 1] - cu_seqlens[r];
    const int32_t w = std::min(window, len);
    const int32_t nr = len - w;
    const int32_t wo = (obs_rows < 0 || obs_rows > len) ? len : obs_rows;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t g = 0; g < n_kv_heads; ++g) {
      std::vector<double> s(len), acc(std::max(nr, 1), 0.0);
      for (int32_t hq = g * G; hq < (g + 1) * G; ++hq)
        for (int32_t i = len - wo; i < len; ++i) {
          const float* qi = q + ((base + i) * n_q_heads + hq) * d;
          double m = -std::numeric_limits<double>::infinity();
          for (int32_t j = 0; j <= i; ++j) {
            s[j] = scale * dot_fd(qi, k + ((base + j) * n_kv_heads + g) * d, d);
            m = std::max(m, s[j]);
          }
          double z = 0.0;
          for (int32_t j = 0; j <= i; ++j) { s[j] = std::exp(s[j] - m); z += s[j]; }
          for (int32_t j = 0; j < nr && j <= i; ++j) acc[j] += s[j] / z;
        }
      for (int32_t j = 0; j < nr; ++j) {
        double v = 0.0;
        const int32_t half = pool > 1 ? pool / 2 : 0;
        for (int32_t jj = j - half; jj <= j + half; ++jj)
          if (jj >= 0 && jj < nr) v += acc[jj];
        c_out[(int64_t)g * T + base + j] = v / (double)(2 * half + 1) / (double)G;
      }
    }
  }
}

// The selection of a policy that uses no scores (attention sinks + recent window, App. A.1 / Table 6): of the
// non-recent keys the first h_keep[r] positions are kept, then the recent window, for every KV head.
int32_t pko_select_sink_recent(int32_t n_req, const int32_t* cu_seqlens, int32_t window, const int32_t* h_keep,
                               const int32_t* cu_kept, int32_t n_kv_heads, int32_t* idx_out) {
  const int64_t K_tot = cu_kept[n_req];
  for (int32_t r = 0; r < n_req; ++r) {
    const int32_t len = cu_seqlens[r + 1] - cu_seqlens[r];
    const int32_t w = std::min(window, len), h = h_keep[r];
    if (h < 0 || h > len - w || cu_kept[r + 1] - cu_kept[r] != h + w) return 1;
    for (int32_t g = 0; g < n_kv_heads; ++g) {
      int32_t* o = idx_out + (int64_t)g * K_tot + cu_kept[r];
      for (int32_t t = 0; t < h; ++t) o[t] = t;
      for (int32_t t = 0; t < w; ++t) o[h + t] = len - w + t;
    }
  }
  return 0;
}

// Spearman's rank correlation of two score vectors (Sec. 3.3, Eq. 7): rho = 1 - 6 sum_j d_j^2 / (n (n^2 - 1)), d_j the
// difference of the two ranks of element j.  The printed upper limit of the sum (j = 0 .. n) has one term too many
// for n elements: the sum runs over the n elements.  Ranks are 1 .. n by descending value; equal values share the
// mean of the ranks they span (the formula is exact only without ties).  n < 2 gives NaN.
double pko_spearman(const double* a, const double* b, int64_t n) {
  if (n < 2) return std::nan("");
  auto ranks = [n](const double* x) {
    std::vector<int64_t> order(n);
    std::iota(order.begin(), order.end(), (int64_t)0);
    std::stable_sort(order.begin(), order.end(), [x](int64_t u, int64_t v) { return x[u] > x[v]; });
    std::vector<double> rk(n);
    for (int64_t p = 0; p < n;) {
      int64_t e = p;
      while (e + 1 < n && x[order[e + 1]] == x[order[p]]) ++e;
      const double mean_rank = 0.5 * (double)(p + e) + 1.0;
      for (int64_t t = p; t <= e; ++t) rk[order[t]] = mean_rank;
      p = e + 1;
    }
    return rk;
  };
  const std::vector<double> ra = ranks(a), rb = ranks(b);
  double sum = 0.0;
  for (int64_t j = 0; j < n; ++j) sum += (ra[j] - rb[j]) * (ra[j] - rb[j]);
  return 1.0 - 6.0 * sum / ((double)n * ((double)n * (double)n - 1.0));
}

// Eq. 3 / Eq. 4 for one layer: S[g, t] = C[g, t] * ||V[t, g, :]||_2.
void pko_vnorm_scores(const double* c /* [H_kv,T] */, const float* v /* [T,H_kv,d] */,
                      int64_t T, int32_t n_kv_heads, int32_t d, double* s_out /* [H_kv,T] */) {
#pragma omp parallel for
  for (int64_t t = 0; t < T; ++t)
    for (int32_t g = 0; g < n_kv_heads; ++g) {
      const float* vv = v + (t * n_kv_heads + g) * d;
      s_out[(int64_t)g * T + t] = c[(int64_t)g * T + t] * std::sqrt(dot_fd(vv, vv, d));
    }
}

// Sec. 3.1 selection for one layer.  For request r and KV head g: the h_keep[r]
// non-recent positions with the largest score (ties: lower position first), written
// in ascending position order, followed by the recent window l-w .. l-1.
// s [H_kv, T]; idx_out [H_kv, K_tot], K_tot = cu_kept[n_req]; positions request-relative.
// kth_out (nullable) [H_kv, n_req]: the h-th largest score (NaN when h == 0).
int32_t pko_select(const double* s, int32_t n_req, const int32_t* cu_seqlens, int32_t window,
                   const int32_t* h_keep, const int32_t* cu_kept, int32_t n_kv_heads,
                   int32_t* idx_out, double* kth_out) {
  const int64_t T = cu_seqlens[n_req];
  const int64_t K_tot = cu_kept[n_req];
  // a budget that asks for more non-recent keys than a request has, or whose kept count is not h + w, is refused
  for (int32_t r = 0; r < n_req; ++r) {
    const int32_t len = cu_seqlens[r + 1] - cu_seqlens[r];
    const int32_t w = std::min(window, len);
    if (h_keep[r] < 0 || h_keep[r] > len - w || cu_kept[r + 1] - cu_kept[r] != h_keep[r] + w) return 1;
  }
  for (int32_t g = 0; g < n_kv_heads; ++g)
    for (int32_t r = 0; r < n_req; ++r) {
      const int64_t base = cu_seqlens[r];
      const int32_t len = cu_seqlens[r + 1] - cu_seqlens[r];
      const int32_t w = std::min(window, len);
      const int32_t nr = len - w;
      const int32_t h = h_keep[r];
      const double* sg = s + (int64_t)g * T + base;
      std::vector<int32_t> order(nr);
      std::iota(order.begin(), order.end(), 0);
      std::stable_sort(order.begin(), order.end(),
                       [&](int32_t a, int32_t b) { return sg[a] > sg[b]; });   // stable: ties keep position order
      std::vector<int32_t> chosen(order.begin(), order.begin() + h);
      std::sort(chosen.begin(), chosen.end());
      int32_t* o = idx_out + (int64_t)g * K_tot + cu_kept[r];
      for (int32_t t = 0; t < h; ++t) o[t] = chosen[t];
      for (int32_t t = 0; t < w; ++t) o[h + t] = nr + t;
      if (kth_out) kth_out[(int64_t)g * n_req + r] = h > 0 ? sg[order[h - 1]] : std::nan("");
    }
  return 0;
}

// Compacted cache of one layer: out[cu_kept[r]+t, g, :] = src[cu_seqlens[r] + idx[g, cu_kept[r]+t], g, :].
// Rows are row_bytes = d * element size bytes; a pure byte copy.
void pko_compact(const uint8_t* src /* [T,H_kv,row_bytes] */, const int32_t* idx /* [H_kv,K_tot] */,
                 int32_t n_req, const int32_t* cu_seqlens, const int32_t* cu_kept,
                 int32_t n_kv_heads, int64_t row_bytes, uint8_t* out /* [K_tot,H_kv,row_bytes] */) {
  const int64_t K_tot = cu_kept[n_req];
  for (int32_t r = 0; r < n_req; ++r)
    for (int32_t t = cu_kept[r]; t < cu_kept[r + 1]; ++t)
      for (int32_t g = 0; g < n_kv_heads; ++g) {
        const int64_t srow = (int64_t)cu_seqlens[r] + idx[(int64_t)g * K_tot + t];
        std::memcpy(out + ((int64_t)t * n_kv_heads + g) * row_bytes,
                    src + (srow * n_kv_heads + g) * row_bytes, (size_t)row_bytes);
      }
}

// Decode step over the compacted cache (Sec. 3.1: later tokens attend to the compressed cache;
// Table 3, decode column).  q [n_req, H, d]: one new query per request; kc, vc [K_tot, H_kv, d]:
// the compact cache of one layer, request r owning rows cu_kept[r] .. cu_kept[r+1]-1; query
// head hq reads KV head hq / G.  out [n_req, H, d] float64; lse [n_req, H] float64 (natural
// log; may be NULL).  A request with no kept key gives out = 0 and lse = -inf.
// scale <= 0 means 1/sqrt(d) (Eq. 1).
void pko_decode(const float* q, const float* kc, const float* vc, int32_t n_req, const int32_t* cu_kept,
                int32_t n_q_heads, int32_t n_kv_heads, int32_t d, double scale, double* out, double* lse) {
  if (scale <= 0.0) scale = 1.0 / std::sqrt((double)d);
  const int32_t G = n_q_heads / n_kv_heads;
  for (int32_t r = 0; r < n_req; ++r) {
    const int64_t j0 = cu_kept[r], j1 = cu_kept[r + 1];
    for (int32_t hq = 0; hq < n_q_heads; ++hq) {
      const int32_t g = hq / G;
      const float* qi = q + ((int64_t)r * n_q_heads + hq) * d;
      double* o = out + ((int64_t)r * n_q_heads + hq) * d;
      for (int32_t c = 0; c < d; ++c) o[c] = 0.0;
      std::vector<double> s((size_t)(j1 - j0));
      double m = -std::numeric_limits<double>::infinity();
      for (int64_t j = j0; j < j1; ++j) {
        s[j - j0] = scale * dot_fd(qi, kc + (j * n_kv_heads + g) * d, d);
        m = std::max(m, s[j - j0]);
      }
      double z = 0.0;
      for (int64_t j = j0; j < j1; ++j) {
        const double e = std::exp(s[j - j0] - m);
        z += e;
        const float* vj = vc + (j * n_kv_heads + g) * d;
        for (int32_t c = 0; c < d; ++c) o[c] += e * (double)vj[c];
      }
      if (j1 > j0)
        for (int32_t c = 0; c < d; ++c) o[c] /= z;
      if (lse) lse[(int64_t)r * n_q_heads + hq] = j1 > j0 ? m + std::log(z) : -std::numeric_limits<double>::infinity();
    }
  }
}

// Budget: w <- min(w, l); k = max(w, floor(keep*l)) capped at l; h = k - w.
void pko_budget(int32_t len, int32_t window, double keep_ratio, int32_t* h_out, int32_t* k_out) {
  const int32_t w = std::min(window, len);
  int32_t k = (int32_t)std::floor(keep_ratio * (double)len);
  k = std::min(len, std::max(w, k));
  *h_out = k - w;
  *k_out = k;
}

}  // extern "C"
