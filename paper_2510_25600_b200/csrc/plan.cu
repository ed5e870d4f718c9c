// Host-side planning for ST-SpAttn prefill (Sec. 3.2): turns the batch shape and the mask
// parameters into per-query-tile lists of kept key tiles, each classified as
//   full    -- every (row, key) pair of the tile is kept: no predicate in the kernel,
//   diag    -- exactly the causal pairs j <= i are kept: only the causal compare,
//   general -- the kernel reads a bit mask (one bit per row and key) stored in the plan.
// Work per query tile is O(rows x intervals): each row's kept keys are a union of a few
// position intervals (prefix + first frames, spans of the current frame, spans or single cells
// of linked earlier frames), accumulated into per-key-tile pair counts; general tiles get their
// bits from the same intervals.  The kernels therefore never evaluate the mask's definition.
#include <algorithm>
#include <cstring>
#include <mutex>
#include <string>
#include <queue>
#include <vector>

#include "common.cuh"

namespace purekv {

static thread_local char g_err[512] = "";
static std::atomic<uint64_t> g_wait_limit_ns{1000ull * 1000ull * 1000ull};

uint64_t wait_limit_ns() { return g_wait_limit_ns.load(std::memory_order_relaxed); }

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

purekv_status check_batch(const purekv_batch* b, bool need_device) {
  PK_REQUIRE(b != nullptr, PUREKV_ERR_INVALID_ARG, "batch is null");
  PK_REQUIRE(b->n_req >= 0 && b->total_tokens >= 0, PUREKV_ERR_INVALID_ARG, "negative batch size");
  PK_REQUIRE(b->h_cu_seqlens != nullptr, PUREKV_ERR_INVALID_ARG, "h_cu_seqlens is null");
  PK_REQUIRE(!need_device || b->cu_seqlens != nullptr || b->n_req == 0 || b->total_tokens == 0, PUREKV_ERR_INVALID_ARG,
             "cu_seqlens (device) is null");
  PK_REQUIRE(b->h_cu_seqlens[0] == 0, PUREKV_ERR_INVALID_ARG, "cu_seqlens[0] must be 0");
  for (int r = 0; r < b->n_req; ++r)
    PK_REQUIRE(b->h_cu_seqlens[r + 1] >= b->h_cu_seqlens[r], PUREKV_ERR_INVALID_ARG,
               "cu_seqlens must be non-decreasing (request %d)", r);
  PK_REQUIRE(b->h_cu_seqlens[b->n_req] == b->total_tokens, PUREKV_ERR_INVALID_ARG,
             "total_tokens %lld != cu_seqlens[n_req] %d", (long long)b->total_tokens,
             b->h_cu_seqlens[b->n_req]);
  return PUREKV_OK;
}

static int64_t align16(int64_t x) { return (x + 15) & ~int64_t(15); }

static purekv_status check_params(const purekv_batch* b, const purekv_st_params* p, purekv_dtype dtype,
                                  int32_t head_dim, int* tile_q, int* tile_k) {
  purekv_status st = check_batch(b, false);
  if (st != PUREKV_OK) return st;
  PK_REQUIRE(p != nullptr, PUREKV_ERR_INVALID_ARG, "params is null");
  PK_REQUIRE(b->h_n_prefix && b->h_n_frames, PUREKV_ERR_INVALID_ARG, "h_n_prefix / h_n_frames is null");
  PK_REQUIRE(p->grid_h >= 1 && p->grid_w >= 1 && p->grid_h <= 32767 && p->grid_w <= 32767,
             PUREKV_ERR_INVALID_ARG, "grid %dx%d out of range", p->grid_h, p->grid_w);
  PK_REQUIRE(p->tile == 16 || p->tile == 32 || p->tile == 64 || p->tile == 128, PUREKV_ERR_UNSUPPORTED,
             "tile %d not in {16,32,64,128}", p->tile);
  PK_REQUIRE(p->anchor_frames >= 0 && p->spatial_radius >= -1 && p->temporal_depth >= -1 &&
                 p->temporal_radius >= -1 && p->temporal_stride >= 1 && p->temporal_stride <= 32767 &&
                 p->temporal_depth <= 32767 && p->local_window >= 0 && p->atrous_dilation >= 0,
             PUREKV_ERR_INVALID_ARG, "mask parameter out of range");
  PK_REQUIRE(dtype == PUREKV_BF16 || dtype == PUREKV_FP32, PUREKV_ERR_INVALID_ARG, "unknown dtype");
  const int64_t n = (int64_t)p->grid_h * p->grid_w;
  for (int r = 0; r < b->n_req; ++r) {
    const int64_t len = b->h_cu_seqlens[r + 1] - b->h_cu_seqlens[r];
    PK_REQUIRE(b->h_n_prefix[r] >= 0 && b->h_n_frames[r] >= 0 && b->h_n_frames[r] <= 32767 &&
                   b->h_n_prefix[r] + b->h_n_frames[r] * n <= len,
               PUREKV_ERR_INVALID_ARG, "request %d: prefix %d + %d frames of %lld tokens exceed length %lld", r,
               b->h_n_prefix[r], b->h_n_frames[r], (long long)n, (long long)len);
  }
  // Tensor-core kernel: 128 query rows per tile, keys per tile = the skip granularity.
  const bool tc = dtype == PUREKV_BF16 && head_dim == 128 && (p->tile == 64 || p->tile == 128);
  *tile_k = p->tile;
  *tile_q = tc ? 128 : std::min(p->tile, 64);  // CUDA-core kernel: at most 64 rows per tile
  return PUREKV_OK;
}

struct Span { int32_t a, b; };  // inclusive request-relative positions

// The status word of calls made without one.  In host code this name is only a stand-in for the symbol: the device
// address comes from cudaGetSymbolAddress, once per device.
static __device__ int32_t g_default_status;

purekv_status default_status_word(int32_t** out) {
  constexpr int kMaxDevices = 64;
  static std::mutex mu;
  static int32_t* ptrs[kMaxDevices] = {};
  int dev = -1;
  PK_CUDA(cudaGetDevice(&dev));
  PK_REQUIRE(dev >= 0 && dev < kMaxDevices, PUREKV_ERR_UNSUPPORTED, "device ordinal %d is beyond %d", dev, kMaxDevices);
  std::lock_guard<std::mutex> lock(mu);
  if (!ptrs[dev]) {
    int32_t* p = nullptr;
    PK_CUDA(cudaGetSymbolAddress((void**)&p, g_default_status));
    PK_REQUIRE(p != nullptr, PUREKV_ERR_CUDA, "cudaGetSymbolAddress returned a null status address");
    ptrs[dev] = p;
  }
  *out = ptrs[dev];
  return PUREKV_OK;
}

}  // namespace purekv

using namespace purekv;

extern "C" {

const char* purekv_version(void) { return "purekv-b200 0.2.0 (sm_100a)"; }

void purekv_set_wait_limit_ns(uint64_t ns) {
  g_wait_limit_ns.store(ns ? ns : 1000ull * 1000ull * 1000ull, std::memory_order_relaxed);
}

void purekv_last_error(char* buf, size_t n) {
  if (!buf || n == 0) return;
  strncpy(buf, g_err, n - 1);
  buf[n - 1] = 0;
}

purekv_status purekv_budget(int32_t len, int32_t window, double keep_ratio, int32_t* h_out, int32_t* k_out) {
  PK_REQUIRE(len >= 0 && window >= 0 && keep_ratio >= 0.0 && h_out && k_out, PUREKV_ERR_INVALID_ARG,
             "purekv_budget: bad argument");
  const int32_t w = std::min(window, len);
  const double kf = keep_ratio * (double)len;
  int32_t k = kf >= (double)len ? len : (int32_t)kf;  // floor of a non-negative value
  k = std::min(len, std::max(w, k));
  *h_out = k - w;
  *k_out = k;
  return PUREKV_OK;
}

// Splits long kept-key lists into chunks and orders the (query tile, head pair, chunk) units by decreasing cost:
// the kernel's n_ctas persistent CTAs start with the first n_ctas units and draw the rest from a counter as they
// finish, so the order is longest-first list scheduling carried out at run time.  The costs also decide how finely
// long lists are cut.  They are in quarters of a 64-key half of a list entry, fitted
// to measured unit times: 4 per present half (5 when the entry carries a bit mask), 6 per unit (query load, pipeline
// fill, epilogue) and 14 more for a chunk of a split list (fp32 partial result written out, and the merge).
//
// With an odd group size the group's last head has no partner; a unit for it alone takes as long as a unit for two
// heads.  Consecutive query tiles of a request whose lists are not split therefore share that head's unit (a twin
// unit, see Unit): the merged lists are appended to `entries`.
static void schedule_units(const std::vector<QTile>& qtiles, std::vector<int2>& entries, int32_t H, int32_t Hkv,
                           int32_t n_ctas,
                           std::vector<Unit>& units, int32_t* n_counters,
                           int64_t* part_slots, int32_t* max_chunks) {
  const int32_t G = H / Hkv, ppg = (G + 1) / 2, n_pairs = Hkv * ppg;
  const bool odd = (G & 1) != 0;
  const int32_t overhead = 6, split_extra = 14;
  const int32_t nq = (int32_t)qtiles.size();
  auto halves = [&](int32_t first, int32_t last) {  // cost of entries [first, last)
    int32_t c = 0;
    for (int32_t i = first; i < last; ++i)
      c += ((((entries[i].x >> 2) & 3) == 3) ? 2 : 1) * ((entries[i].x & 3) == kTileGeneral ? 5 : 4);
    return c;
  };
  // The union of two runs of entries (of two query tiles' lists) in key-tile order: its cost and length; the entry
  // pairs go to `out` if given.
  auto merge_lists = [&](int32_t ia, int32_t ea, int32_t ib, int32_t eb, std::vector<int2>* out, int32_t* count) {
    int32_t cost = 0, n = 0;
    while (ia < ea || ib < eb) {
      const int32_t ka = ia < ea ? (entries[ia].x >> 4) : INT32_MAX, kb = ib < eb ? (entries[ib].x >> 4) : INT32_MAX;
      const int32_t kt = std::min(ka, kb);
      const int2 none = make_int2((kt << 4) | kTileNone, -1);
      const int2 xa = ka == kt ? entries[ia++] : none, xb = kb == kt ? entries[ib++] : none;
      const bool both = (((xa.x | xb.x) >> 2) & 3) == 3;
      const bool bits = (xa.x & 3) == kTileGeneral || (xb.x & 3) == kTileGeneral;
      cost += (both ? 2 : 1) * (bits ? 5 : 4);
      if (out) { out->push_back(xa); out->push_back(xb); }
      ++n;
    }
    *count = n;
    return cost;
  };
  auto chunks_of = [&](const QTile& q, int32_t l_max) { return std::max(1, (q.entry_count + l_max - 1) / l_max); };
  // chunk c of nch of a tile's list, as a range of entries[]
  auto chunk_range = [&](const QTile& q, int32_t c, int32_t nch, int32_t* first, int32_t* last) {
    *first = q.entry_begin + (int32_t)((int64_t)q.entry_count * c / nch);
    *last = q.entry_begin + (int32_t)((int64_t)q.entry_count * (c + 1) / nch);
  };
  // partner[i]: the tile that shares tile i's odd-head units (i leads the twin), -2 if tile i is the second of a
  // twin, -1 if it stays alone.  Twins have the same number of chunks, and a merged chunk may be a quarter longer
  // than the cap on a chunk.
  std::vector<int32_t> partner;
  auto find_twins = [&](int32_t l_max) {
    partner.assign((size_t)nq, -1);
    if (!odd) return;
    for (int32_t i = 0; i + 1 < nq; ++i) {
      const QTile &a = qtiles[i], &b = qtiles[i + 1];
      const int32_t nch = chunks_of(a, l_max);
      if (partner[i] != -1 || a.req_start != b.req_start || nch != chunks_of(b, l_max)) continue;
      bool fits = true;
      for (int32_t c = 0; c < nch && fits; ++c) {
        int32_t a0, a1, b0, b1, n = 0;
        chunk_range(a, c, nch, &a0, &a1);
        chunk_range(b, c, nch, &b0, &b1);
        merge_lists(a0, a1, b0, b1, nullptr, &n);
        fits = n <= l_max + l_max / 4;
      }
      if (!fits) continue;
      partner[i] = i + 1;
      partner[i + 1] = -2;
    }
  };
  struct Item { Unit u; int32_t cost; };
  std::vector<Item> items;
  std::vector<int2> twin_entries;
  std::vector<int32_t> part_of, counter_of;  // per query tile: first workspace slot and merge counter, -1 if unsplit
  int32_t counters = 0, mc = 1;
  int64_t slots = 0;
  // the units when no chunk of a list may be longer than l_max entries
  auto make_items = [&](int32_t l_max) {
    items.clear();
    twin_entries.clear();
    counters = 0; mc = 1; slots = 0;
    find_twins(l_max);
    part_of.assign((size_t)nq, -1);
    counter_of.assign((size_t)nq, -1);
    for (int32_t qi = 0; qi < nq; ++qi) {
      const int32_t nch = chunks_of(qtiles[qi], l_max);
      mc = std::max(mc, nch);
      if (nch > 1) {
        part_of[qi] = (int32_t)slots;
        counter_of[qi] = counters;
        slots += nch;
        counters += H;
      }
    }
    for (int32_t qi = 0; qi < nq; ++qi) {
      const QTile& q = qtiles[qi];
      const int32_t nch = chunks_of(q, l_max);
      for (int32_t c = 0; c < nch; ++c) {
        int32_t a, e;
        chunk_range(q, c, nch, &a, &e);
        const int32_t cost = halves(a, e) + overhead + (nch > 1 ? split_extra : 0);
        for (int32_t pr = 0; pr < n_pairs; ++pr) {
          if (partner[qi] != -1 && pr % ppg == ppg - 1) continue;  // the odd head goes into a twin unit
          Unit u = {};
          u.q_start = q.q_start; u.q_rows = q.q_rows; u.req_start = q.req_start;
          u.ent_begin = a; u.ent_count = e - a;
          u.pair = pr; u.chunk = c; u.n_chunks = nch;
          u.part_base = part_of[qi]; u.counter_base = counter_of[qi];
          u.part_base1 = u.counter_base1 = -1;
          items.push_back({u, cost});
        }
        if (partner[qi] >= 0) {
          const QTile& q1 = qtiles[partner[qi]];
          int32_t a1, e1, n = 0;
          chunk_range(q1, c, nch, &a1, &e1);
          const int32_t at = (int32_t)(entries.size() + twin_entries.size());
          const int32_t cost2 = merge_lists(a, e, a1, e1, &twin_entries, &n) + overhead + (nch > 1 ? split_extra : 0);
          for (int32_t g = 0; g < Hkv; ++g) {
            Unit u = {};
            u.q_start = q.q_start; u.q_rows = q.q_rows; u.req_start = q.req_start;
            u.q_start1 = q1.q_start; u.q_rows1 = q1.q_rows;
            u.ent_begin = at; u.ent_count = n;
            u.pair = g * ppg + ppg - 1; u.chunk = c; u.n_chunks = nch;
            u.part_base = part_of[qi]; u.counter_base = counter_of[qi];
            u.part_base1 = part_of[partner[qi]]; u.counter_base1 = counter_of[partner[qi]];
            items.push_back({u, cost2});
          }
        }
      }
    }
    std::stable_sort(items.begin(), items.end(), [](const Item& x, const Item& y) { return x.cost > y.cost; });
  };
  // the time the last CTA ends when the CTAs draw units of these costs in decreasing order, each as it becomes free
  std::vector<int32_t> costs;
  auto makespan = [&](int32_t l_max) {
    costs.clear();
    find_twins(l_max);
    for (int32_t qi = 0; qi < nq; ++qi) {
      const QTile& q = qtiles[qi];
      const int32_t nch = chunks_of(q, l_max);
      for (int32_t c = 0; c < nch; ++c) {
        int32_t a, e;
        chunk_range(q, c, nch, &a, &e);
        const int32_t extra = overhead + (nch > 1 ? split_extra : 0);
        costs.insert(costs.end(), (size_t)(partner[qi] != -1 ? n_pairs - Hkv : n_pairs), halves(a, e) + extra);
        if (partner[qi] >= 0) {
          int32_t a1, e1, n = 0;
          chunk_range(qtiles[partner[qi]], c, nch, &a1, &e1);
          costs.insert(costs.end(), (size_t)Hkv, merge_lists(a, e, a1, e1, nullptr, &n) + extra);
        }
      }
    }
    std::sort(costs.begin(), costs.end(), std::greater<int32_t>());
    std::priority_queue<int64_t, std::vector<int64_t>, std::greater<int64_t>> load;
    for (int32_t c = 0; c < n_ctas; ++c) load.push(0);
    int64_t end = 0;
    for (int32_t cost : costs) {
      const int64_t t = load.top() + cost;
      load.pop();
      load.push(t);
      end = std::max(end, t);
    }
    return end;
  };
  // Splitting shortens the units the CTAs end on but costs a partial result and a merge per chunk.  With few units
  // per CTA the trade is decided by trying: the cap on a chunk's length that ends soonest under the cost model wins.
  // With many units the ends even out by themselves and only the very longest lists are cut.
  int32_t l_best = 64;
  if ((int64_t)qtiles.size() * n_pairs < 12 * (int64_t)n_ctas) {
    int64_t t_best = -1;
    for (int32_t l_max : {64, 24, 12, 9, 7, 5}) {
      const int64_t t = makespan(l_max);
      if (t_best < 0 || t <= t_best) { t_best = t; l_best = l_max; }  // on a tie the finer cut
    }
  }
  make_items(l_best);
  entries.insert(entries.end(), twin_entries.begin(), twin_entries.end());
  units.clear();
  for (const Item& it : items) units.push_back(it.u);
  *n_counters = counters;
  *part_slots = slots * H;
  *max_chunks = mc;
}

static purekv_status build_plan(const purekv_batch* b, const purekv_st_params* p, purekv_dtype dtype,
                                int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, int32_t n_ctas,
                                purekv_plan_info* info, std::vector<uint8_t>& host) {
  int tq, gk;  // rows per query tile; skip granularity in keys (the mask parameter `tile`)
  purekv_status st = check_params(b, p, dtype, head_dim, &tq, &gk);
  if (st != PUREKV_OK) return st;
  // The tensor-core kernel always works on 128-key entries; with a 64-key skip granularity an entry carries a
  // 2-bit mask of the halves that hold kept pairs, and an absent half is neither loaded nor computed.
  const int32_t tk = tq == 128 ? 128 : gk;  // keys per list entry
  const int32_t hpe = tk / gk;              // key blocks of the skip granularity per entry (1 or 2)
  PK_REQUIRE(info, PUREKV_ERR_INVALID_ARG, "info is null");
  PK_REQUIRE(n_q_heads >= 1 && n_kv_heads >= 1 && n_q_heads % n_kv_heads == 0 && n_q_heads <= 65535,
             PUREKV_ERR_INVALID_ARG, "n_q_heads %d must be a positive multiple of n_kv_heads %d", n_q_heads,
             n_kv_heads);
  PK_REQUIRE(n_ctas >= 0 && n_ctas <= 4096, PUREKV_ERR_INVALID_ARG, "n_ctas %d outside [0, 4096]", n_ctas);
  if (n_ctas == 0) n_ctas = 148;  // one persistent CTA per SM of a B200
  const bool dense = (p->flags & PUREKV_FLAG_DENSE_CAUSAL) != 0;
  const int32_t gw = p->grid_w, gh = p->grid_h, n = gw * gh;
  const int64_t T = b->total_tokens;
  const int32_t wpr = std::max(1, tk / 32);  // mask words per row of a general tile

  std::vector<QTile> qtiles;
  std::vector<int2> entries;
  std::vector<uint32_t> masks;
  memset(info, 0, sizeof(*info));

  std::vector<int64_t> cnt, diff, cg;  // kept pairs per gk-key block of the current query tile
  std::vector<Span> spans, row_spans, merged;
  std::vector<char> blk_kept;
  const bool coarse = (p->flags & PUREKV_FLAG_COARSE_BLOCKS) != 0 && !dense;
  std::vector<int32_t> row_off;
  for (int r = 0; r < b->n_req; ++r) {
    const int32_t base = b->h_cu_seqlens[r];
    const int32_t len = b->h_cu_seqlens[r + 1] - base;
    const int32_t npre = b->h_n_prefix[r], nfr = b->h_n_frames[r];
    const int32_t vis_end = npre + nfr * n;
    const int32_t nkt = (len + gk - 1) / gk + 2;
    cnt.assign((size_t)nkt + 2, 0);
    diff.assign((size_t)nkt + 3, 0);
    cg.assign((size_t)nkt + 3, 0);
    const int32_t anchor_end = (int32_t)std::min<int64_t>(vis_end, npre + (int64_t)p->anchor_frames * n);  // exclusive
    // the token-level mask of row i as disjoint ascending spans of kept key positions
    auto token_spans = [&](int32_t i, std::vector<Span>& out) {
      out.clear();
      const bool visual = i >= npre && i < vis_end;
      if (dense || !visual) {
        out.push_back({0, i});  // text rows and the dense mask: plain causal
        return;
      }
      spans.clear();
      if (anchor_end > 0) spans.push_back({0, std::min(i, anchor_end - 1)});  // prefix + first frame(s)
      const int32_t f = (i - npre) / n, c = (i - npre) % n, y = c / gw, x = c % gw;
      const int32_t fs = npre + f * n;
      if (p->spatial_radius < 0) {
        spans.push_back({fs, i});  // the current frame, causal
      } else {
        const int32_t rr = p->spatial_radius;
        for (int32_t yy = std::max(0, y - rr); yy <= y; ++yy) {
          const int32_t xa = std::max(0, x - rr), xb = yy == y ? x : std::min(gw - 1, x + rr);
          spans.push_back({fs + yy * gw + xa, fs + yy * gw + xb});
        }
      }
      for (int32_t m = 1;; ++m) {  // linked earlier frames: the corresponding cell (or a window / the frame)
        const int64_t fj = (int64_t)f - (int64_t)m * p->temporal_stride;
        if (fj < 0 || (p->temporal_depth >= 0 && m > p->temporal_depth)) break;
        const int32_t fjs = npre + (int32_t)fj * n;
        if (p->temporal_radius < 0) {
          spans.push_back({fjs, fjs + n - 1});
        } else {
          const int32_t rr = p->temporal_radius;
          for (int32_t yy = std::max(0, y - rr); yy <= std::min(gh - 1, y + rr); ++yy)
            spans.push_back({fjs + yy * gw + std::max(0, x - rr), fjs + yy * gw + std::min(gw - 1, x + rr)});
        }
      }
      if (p->local_window > 0) spans.push_back({std::max(npre, i - p->local_window + 1), i});  // the most recent positions
      if (p->atrous_dilation > 0)                                                             // every D-th position back
        for (int32_t j = i; j >= npre; j -= p->atrous_dilation) spans.push_back({j, j});
      std::sort(spans.begin(), spans.end(), [](const Span& u, const Span& v) { return u.a < v.a; });
      int32_t ca = spans[0].a, cb = spans[0].b;
      for (size_t s = 1; s < spans.size(); ++s) {
        if (spans[s].a <= cb + 1) cb = std::max(cb, spans[s].b);
        else { out.push_back({ca, cb}); ca = spans[s].a; cb = spans[s].b; }
      }
      out.push_back({ca, cb});
    };
    int32_t cached_rb = -1;          // block of rows whose kept key blocks are in blk_kept (coarse masks)
    for (int32_t q0 = 0; q0 < len; q0 += tq) {
      const int32_t q1 = std::min(len, q0 + tq);  // exclusive
      const int32_t kt_hi = (q1 - 1) / tk;        // last list entry a causal mask reaches
      const int32_t kg_hi = (q1 - 1) / gk;        // last gk-key block a causal mask reaches
      std::fill(cnt.begin(), cnt.begin() + kg_hi + 3, 0);
      std::fill(diff.begin(), diff.begin() + kg_hi + 4, 0);
      row_spans.clear();
      row_off.assign(1, 0);
      auto add_span = [&](int32_t a, int32_t bb) {  // inclusive, a <= bb
        row_spans.push_back({a, bb});
        const int32_t ta = a / gk, tb = bb / gk;
        if (ta == tb) { cnt[ta] += bb - a + 1; return; }
        cnt[ta] += (ta + 1) * gk - a;
        cnt[tb] += bb - tb * gk + 1;
        diff[ta + 1] += gk;
        diff[tb] -= gk;
      };
      // each row's kept keys as disjoint ascending spans (Sec. 3.2; App. A.3 for the local and atrous terms)
      for (int32_t i = q0; i < q1; ++i) {
        if (!coarse) {
          token_spans(i, merged);
          for (const Span& sp : merged) add_span(sp.a, sp.b);
        } else {
          // block-level widening: the key blocks in which any row of this row's block keeps a pair (found once per
          // block of rows), each taken whole up to the diagonal
          const int32_t rb = i / gk;
          if (rb != cached_rb) {
            cached_rb = rb;
            const int32_t r_hi = std::min(len, rb * gk + gk);
            blk_kept.assign((size_t)(r_hi - 1) / gk + 1, 0);
            for (int32_t ii = rb * gk; ii < r_hi; ++ii) {
              token_spans(ii, merged);
              for (const Span& sp : merged)
                for (int32_t kb = sp.a / gk; kb <= sp.b / gk; ++kb) blk_kept[kb] = 1;
            }
          }
          for (int32_t kb = 0; kb <= i / gk; ++kb) {
            if (!blk_kept[kb]) continue;
            int32_t ke = kb;
            while (ke + 1 <= i / gk && blk_kept[ke + 1]) ++ke;
            add_span(kb * gk, std::min(ke * gk + gk - 1, i));
            kb = ke;
          }
        }
        row_off.push_back((int32_t)row_spans.size());
      }
      QTile qt;
      qt.q_start = base + q0;
      qt.q_rows = q1 - q0;
      qt.req_start = base;
      qt.req_len = len;
      qt.entry_begin = (int32_t)entries.size();
      qt.pad[0] = qt.pad[1] = 0;
      int64_t run = 0;
      for (int32_t kg = 0; kg <= kg_hi + 1; ++kg) {
        run += diff[kg];
        cg[kg] = cnt[kg] + run;
      }
      info->tiles_causal += kg_hi + 1;
      for (int32_t kt = 0; kt <= kt_hi; ++kt) {
        int64_t c = 0;
        int32_t half_mask = 0;
        for (int32_t hh = 0; hh < hpe; ++hh) {
          const int32_t kg = kt * hpe + hh;
          if (kg <= kg_hi && cg[kg] > 0) { c += cg[kg]; half_mask |= 1 << hh; info->tiles_kept++; }
        }
        if (c == 0) continue;
        if (hpe == 1) half_mask = 3;  // one block per entry: both bits set by convention
        const int32_t j0 = kt * tk;
        const int64_t full = (int64_t)(q1 - q0) * tk;
        int64_t causal = full;  // pairs with j <= i inside this tile
        if (j0 + tk - 1 > q0) {
          causal = 0;
          for (int32_t i = q0; i < q1; ++i) causal += std::max(0, std::min(tk, i - j0 + 1));
        }
        int32_t cls = kTileGeneral, mask_at = -1;
        if (c == full && j0 + tk <= len) cls = kTileFull;
        else if (c == causal) cls = kTileDiag;
        if (cls == kTileGeneral) {
          // one bit per (row, key) of the tile, rows past q_rows stay zero
          PK_REQUIRE(masks.size() + (size_t)tq * wpr < (size_t)INT32_MAX, PUREKV_ERR_UNSUPPORTED,
                     "mask table exceeds 2^31 words");
          mask_at = (int32_t)masks.size();
          masks.resize(masks.size() + (size_t)tq * wpr, 0u);
          uint32_t* mw = masks.data() + mask_at;
          for (int32_t i = q0; i < q1; ++i)
            for (int32_t s = row_off[i - q0]; s < row_off[i - q0 + 1]; ++s) {
              const int32_t a = std::max(row_spans[s].a, j0), bb = std::min(row_spans[s].b, j0 + tk - 1);
              if (a > bb) continue;
              const int32_t lo = a - j0, hi = bb - j0;  // bit range inside the tile row
              uint32_t* rw = mw + (i - q0) * wpr;
              for (int32_t w = lo >> 5; w <= (hi >> 5); ++w) {
                const int32_t b0 = std::max(lo - 32 * w, 0), b1 = std::min(hi - 32 * w, 31);
                rw[w] |= (b1 - b0 == 31) ? 0xFFFFFFFFu : (((1u << (b1 - b0 + 1)) - 1u) << b0);
              }
            }
        }
        entries.push_back(make_int2((kt << 4) | (half_mask << 2) | cls, mask_at));
        info->pairs_kept += c;
        (cls == kTileFull ? info->tiles_full : cls == kTileDiag ? info->tiles_diag : info->tiles_general)++;
      }
      qt.entry_count = (int32_t)entries.size() - qt.entry_begin;
      info->max_list = std::max(info->max_list, qt.entry_count);
      qtiles.push_back(qt);
    }
  }
  const int32_t nq = (int32_t)qtiles.size();
  std::vector<int32_t> order((size_t)nq);
  for (int32_t i = 0; i < nq; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(),
                   [&](int32_t u, int32_t v) { return qtiles[u].entry_count > qtiles[v].entry_count; });

  // tensor-core plans carry the persistent kernel's schedule
  std::vector<Unit> units;
  int32_t n_counters = 0, max_chunks = 1;
  int64_t part_slots = 0;
  if (tq == 128 && nq > 0) {
    schedule_units(qtiles, entries, n_q_heads, n_kv_heads, n_ctas, units, &n_counters, &part_slots, &max_chunks);
  } else {
    n_ctas = 0;
  }

  PlanHeader h;
  memset(&h, 0, sizeof(h));
  h.magic = kPlanMagic;
  h.tile_q = tq;
  h.tile_k = tk;
  h.n_qtiles = nq;
  h.total_tokens = T;
  h.n_entries = (int64_t)entries.size();
  h.n_mask_words = (int64_t)masks.size();
  h.words_per_row = wpr;
  h.off_qtiles = align16(sizeof(PlanHeader));
  h.off_order = h.off_qtiles + align16((int64_t)nq * sizeof(QTile));
  h.off_entries = h.off_order + align16((int64_t)nq * 4);
  h.off_masks = h.off_entries + align16(h.n_entries * 8);
  h.n_ctas = units.empty() ? 0 : n_ctas;
  h.n_units = (int32_t)units.size();
  h.n_counters = n_counters;
  h.n_q_heads = n_q_heads;
  h.n_kv_heads = n_kv_heads;
  h.part_slots = part_slots;
  h.off_units = h.off_masks + align16(h.n_mask_words * 4);
  h.off_counters = h.off_units + align16((int64_t)h.n_units * sizeof(Unit));
  // the merge counters, then the kernel's two scheduling counters; all start at zero and the kernel leaves them so
  const int64_t total = h.off_counters + align16(((int64_t)n_counters + 2) * 4);

  host.assign((size_t)total, 0);
  memcpy(host.data(), &h, sizeof(h));
  if (nq) memcpy(host.data() + h.off_qtiles, qtiles.data(), (size_t)nq * sizeof(QTile));
  if (nq) memcpy(host.data() + h.off_order, order.data(), (size_t)nq * 4);
  if (!entries.empty()) memcpy(host.data() + h.off_entries, entries.data(), entries.size() * 8);
  if (!masks.empty()) memcpy(host.data() + h.off_masks, masks.data(), masks.size() * 4);
  if (!units.empty()) {
    memcpy(host.data() + h.off_units, units.data(), units.size() * sizeof(Unit));
  }

  info->tile_q = tq;
  info->tile_k = gk;
  info->n_qtiles = nq;
  info->bytes_used = total;
  info->dtype = (int32_t)dtype;
  info->head_dim = head_dim;
  info->n_q_heads = n_q_heads;
  info->n_kv_heads = n_kv_heads;
  info->n_ctas = h.n_ctas;
  info->n_units = h.n_units;
  info->max_chunks = max_chunks;
  info->ws_bytes = part_slots * kPartFloats * (int64_t)sizeof(float);
  return PUREKV_OK;
}

size_t purekv_plan_bytes(const purekv_batch* b, const purekv_st_params* p, purekv_dtype dtype, int32_t head_dim,
                         int32_t n_q_heads, int32_t n_kv_heads, int32_t n_ctas) {
  purekv_plan_info info;
  std::vector<uint8_t> host;
  if (build_plan(b, p, dtype, head_dim, n_q_heads, n_kv_heads, n_ctas, &info, host) != PUREKV_OK) return 0;
  return host.size();
}

purekv_status purekv_plan_build_host(const purekv_batch* b, const purekv_st_params* p, purekv_dtype dtype,
                                     int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, int32_t n_ctas,
                                     void* h_plan, size_t plan_bytes, purekv_plan_info* info) {
  PK_REQUIRE(h_plan, PUREKV_ERR_INVALID_ARG, "h_plan is null");
  std::vector<uint8_t> host;
  purekv_status st = build_plan(b, p, dtype, head_dim, n_q_heads, n_kv_heads, n_ctas, info, host);
  if (st != PUREKV_OK) return st;
  PK_REQUIRE(host.size() <= plan_bytes, PUREKV_ERR_WORKSPACE, "plan needs %zu bytes, buffer has %zu", host.size(),
             plan_bytes);
  memcpy(h_plan, host.data(), host.size());
  return PUREKV_OK;
}

purekv_status purekv_plan_build(const purekv_batch* b, const purekv_st_params* p, purekv_dtype dtype,
                                int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, int32_t n_ctas, void* plan,
                                size_t plan_bytes, purekv_plan_info* info, void* stream) {
  PK_REQUIRE(plan, PUREKV_ERR_INVALID_ARG, "plan is null");
  std::vector<uint8_t> host;
  purekv_status st = build_plan(b, p, dtype, head_dim, n_q_heads, n_kv_heads, n_ctas, info, host);
  if (st != PUREKV_OK) return st;
  PK_REQUIRE(host.size() <= plan_bytes, PUREKV_ERR_WORKSPACE, "plan needs %zu bytes, buffer has %zu", host.size(),
             plan_bytes);
  cudaStream_t s = (cudaStream_t)stream;
  PK_CUDA(cudaMemcpyAsync(plan, host.data(), host.size(), cudaMemcpyHostToDevice, s));
  PK_CUDA(cudaStreamSynchronize(s));
  return PUREKV_OK;
}

purekv_status purekv_poll_status(const int32_t* status, int32_t* h_out, void* stream) {
  cudaStream_t s = (cudaStream_t)stream;
  PK_CUDA(cudaStreamSynchronize(s));
  int32_t v = 0;
  if (status) {
    PK_CUDA(cudaMemcpy(&v, status, sizeof(v), cudaMemcpyDeviceToHost));
  } else {
    // the library's own word, used by calls made with status == NULL: report it and clear it, so that one expired
    // wait does not block every later call of that kind
    int32_t* own = nullptr;
    purekv_status st = default_status_word(&own);
    if (st != PUREKV_OK) return st;
    PK_CUDA(cudaMemcpy(&v, own, sizeof(v), cudaMemcpyDeviceToHost));
    if (v != 0) PK_CUDA(cudaMemset(own, 0, sizeof(v)));
  }
  if (h_out) *h_out = v;
  PK_REQUIRE(v != (int32_t)PUREKV_ERR_BAD_PLAN, PUREKV_ERR_BAD_PLAN,
             "device status word is %d: a kernel refused the plan it was handed", v);
  PK_REQUIRE(v == 0, PUREKV_ERR_TIMEOUT, "device status word is %d: a bounded device-side wait expired", v);
  return PUREKV_OK;
}

}  // extern "C"
