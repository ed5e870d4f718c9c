// purekv_select_topk: V-norm weighting (Eq. 3 / Eq. 4) and budgeted top-h selection (Sec. 3.1).
//
// Two paths.  With few (request, head, layer) segments, vnorm_score_kernel streams V once over the whole GPU (the
// only large traffic of this step): a warp owns 32 consecutive (token, head) rows, each half-warp reads one
// 16-byte-chunked row per step and reduces the squared norm with shuffles; select_kernel then handles one segment
// per CTA.  With many segments one CTA does both for its segment and the scores never leave the SM.  The selection
// is a 4 x 8-bit MSB-first radix select over the fp32 bit patterns (keys staged in shared memory) that finds the
// h-th largest score, then a block-scan compaction that emits the chosen positions in ascending order; among
// scores equal to the threshold the lowest positions win, so the result is deterministic.
#include <algorithm>

#include "common.cuh"

namespace purekv {

template <typename T>
struct Chunk;  // one 16-byte load
template <>
struct Chunk<float> {
  static __device__ __forceinline__ float sumsq(uint4 u) {
    const float a = __uint_as_float(u.x), b = __uint_as_float(u.y), c = __uint_as_float(u.z),
                d = __uint_as_float(u.w);
    return a * a + b * b + c * c + d * d;
  }
};
template <>
struct Chunk<__nv_bfloat16> {
  static __device__ __forceinline__ float sumsq(uint4 u) {
    float s = 0.f;
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
      s = fmaf(lo, lo, s);
      s = fmaf(hi, hi, s);
    }
    return s;
  }
};

// grid: one dimension, at most 3 CTAs per SM (a single full wave whatever the number of layers and heads); the warps
// stride over blocks of 32 consecutive (token, head) rows of a layer, i.e. over contiguous memory.
// block: 256 threads = 8 warps.
template <typename T>
__global__ void __launch_bounds__(256, 3) vnorm_score_kernel(const uint4* __restrict__ v, int64_t layer_stride_c,
                                                          const float* __restrict__ c, int64_t n_tokens,
                                                          int32_t n_kv_heads, int32_t n_layers, int32_t chunks_per_row,
                                                          float* __restrict__ s_out) {
  const int32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t n_rows = n_tokens * n_kv_heads;  // rows of one layer, row = token * n_kv_heads + head
  const int64_t n_blocks = (n_rows + 31) / 32;
  const int64_t n_items = n_blocks * n_layers;
  for (int64_t item = (int64_t)blockIdx.x * 8 + warp; item < n_items; item += (int64_t)gridDim.x * 8) {
    const int64_t blk = item % n_blocks;
    const int32_t layer = (int32_t)(item / n_blocks);
    const uint4* vl = v + layer * layer_stride_c;
    const int64_t r0 = blk * 32;
    float mine = 0.f;
    if (chunks_per_row == 16) {
      // 256-byte rows: a half-warp covers one row per step, 16 steps cover 32 rows (8 KB of contiguous memory).
      const int32_t half = lane >> 4, ch = lane & 15;
      float part[16];
      // all 16 loads are issued before the first use (volatile asm keeps them ahead of the arithmetic): with the 8 KB
      // of a warp in flight at once, three CTAs per SM keep enough bytes outstanding to stream V near the DRAM rate
      uint4 buf[16];
#pragma unroll
      for (int it = 0; it < 16; ++it) {
        const int64_t r = min(r0 + it * 2 + half, n_rows - 1);  // rows past the end re-read the last one; never stored
        const uint4* p = vl + r * 16 + ch;
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(buf[it].x), "=r"(buf[it].y), "=r"(buf[it].z), "=r"(buf[it].w) : "l"(p));
      }
#pragma unroll
      for (int it = 0; it < 16; ++it) part[it] = Chunk<T>::sumsq(buf[it]);
#pragma unroll
      for (int it = 0; it < 16; ++it) {
        float p = part[it];
        p += __shfl_xor_sync(0xffffffffu, p, 8);
        p += __shfl_xor_sync(0xffffffffu, p, 4);
        p += __shfl_xor_sync(0xffffffffu, p, 2);
        p += __shfl_xor_sync(0xffffffffu, p, 1);
        // lanes 0..15 now hold row 2*it's sum, lanes 16..31 row 2*it+1's; lane L keeps row L
        const float v0 = __shfl_sync(0xffffffffu, p, 0), v1 = __shfl_sync(0xffffffffu, p, 16);
        if (lane == it * 2) mine = v0;
        if (lane == it * 2 + 1) mine = v1;
      }
    } else {
      // generic row length: one row per lane, sequential chunks
      const int64_t r = r0 + lane;
      if (r < n_rows) {
        const uint4* row = vl + r * chunks_per_row;
        for (int32_t ch = 0; ch < chunks_per_row; ++ch) mine += Chunk<T>::sumsq(__ldg(row + ch));
      }
    }
    const int64_t r = r0 + lane;
    if (r < n_rows) {
      const int64_t t = r / n_kv_heads;
      const int32_t g = (int32_t)(r % n_kv_heads);
      s_out[((int64_t)layer * n_kv_heads + g) * n_tokens + t] = __ldg(c + (int64_t)g * n_tokens + t) * sqrtf(mine);
    }
  }
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // see select_kernel
}

__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kSelThreads = 512;

// What the selecting CTA needs to also gather its segment's kept rows into the compact cache (Sec. 3.1: the selection
// feeds the compressed cache directly); k_src == nullptr: selection only.  Rows are `cpr` 16-byte chunks; layer
// strides in chunks.
struct Gather {
  const uint4 *k_src, *v_src;
  uint4 *k_dst, *v_dst;
  int64_t src_layer_stride_c, dst_layer_stride_c;
  int32_t cpr;
};

// One CTA per (request, KV head, layer).  FUSED = false: the scores come from `s` (written by vnorm_score_kernel).
// FUSED = true: the CTA first streams its own segment of V (256-byte rows), forms S = C * ||V|| into shared memory
// (and into s_out if asked), and selects from there, so V is the only large read and S never makes a round trip;
// used when there are enough segments to keep every SM streaming.
template <bool FUSED, typename T, bool GATHER = false>
__global__ void __launch_bounds__(kSelThreads) select_kernel(const float* __restrict__ s, int64_t n_tokens,
                                                             const int32_t* __restrict__ cu_seqlens,
                                                             const int32_t* __restrict__ cu_kept,
                                                             const int32_t* __restrict__ keep, int32_t window,
                                                             int32_t k_tot, int32_t n_kv_heads,
                                                             int32_t* __restrict__ idx_out, const uint4* __restrict__ v,
                                                             int64_t layer_stride_c, const float* __restrict__ c,
                                                             float* __restrict__ s_out, Gather ga) {
  extern __shared__ __align__(16) uint32_t skeys[];  // order keys of the segment's non-recent scores
  __shared__ int32_t hist[256];
  __shared__ uint32_t sh_prefix;
  __shared__ int32_t sh_need;
  __shared__ int32_t warp_gt[32], warp_eq[32];
  __shared__ int32_t carry_eq;

  const int32_t r = blockIdx.x, g = blockIdx.y, layer = blockIdx.z;
  // launched with programmatic stream serialization behind vnorm_score_kernel, which releases its dependents only
  // when its own work is done: the launch latency overlaps that kernel's tail, and its scores are complete and
  // visible from here on (no effect in an ordinary launch)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int32_t base = cu_seqlens[r];
  const int32_t len = cu_seqlens[r + 1] - base;
  const int32_t w = min(window, len);
  const int32_t nr = len - w;
  const int32_t h = keep[r];
  const float* seg = s + ((int64_t)layer * n_kv_heads + g) * n_tokens + base;
  int32_t* out = idx_out + ((int64_t)layer * n_kv_heads + g) * k_tot + cu_kept[r];
  const int32_t tid = threadIdx.x;

  for (int32_t t = tid; t < w; t += kSelThreads) out[h + t] = nr + t;  // the recent window
  if constexpr (FUSED) {
    // a half-warp reads one 256-byte row per step (16 x 16 bytes), 16 rows in flight per thread
    const uint4* vl = v + layer * layer_stride_c;
    const float* cg = c + (int64_t)g * n_tokens + base;
    float* so = s_out ? s_out + ((int64_t)layer * n_kv_heads + g) * n_tokens + base : nullptr;
    const int32_t lane = tid & 31, wrp = tid >> 5, half = lane >> 4, ch = lane & 15;
    const int32_t n_score = so ? len : nr;  // the window's scores are 0 by definition and only matter for s_out
    for (int32_t t0 = wrp * 32; t0 < n_score; t0 += (kSelThreads / 32) * 32) {
      // as in vnorm_score_kernel: the 16 row loads of the trip are issued before the first is used
      float part[16];
      uint4 buf[16];
#pragma unroll
      for (int it = 0; it < 16; ++it) {
        const int32_t t = min(t0 + it * 2 + half, n_score - 1);  // rows past the end re-read the last one; never stored
        const uint4* p = vl + ((int64_t)(base + t) * n_kv_heads + g) * 16 + ch;
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(buf[it].x), "=r"(buf[it].y), "=r"(buf[it].z), "=r"(buf[it].w) : "l"(p));
      }
#pragma unroll
      for (int it = 0; it < 16; ++it) part[it] = Chunk<T>::sumsq(buf[it]);
      float mine = 0.f;
#pragma unroll
      for (int it = 0; it < 16; ++it) {
        float p = part[it];
        p += __shfl_xor_sync(0xffffffffu, p, 8);
        p += __shfl_xor_sync(0xffffffffu, p, 4);
        p += __shfl_xor_sync(0xffffffffu, p, 2);
        p += __shfl_xor_sync(0xffffffffu, p, 1);
        const float v0 = __shfl_sync(0xffffffffu, p, 0), v1 = __shfl_sync(0xffffffffu, p, 16);
        if (lane == it * 2) mine = v0;
        if (lane == it * 2 + 1) mine = v1;
      }
      const int32_t t = t0 + lane;
      if (t < n_score) {
        const float sc = __ldg(cg + t) * sqrtf(mine);
        if (so) so[t] = sc;
        if (t < nr) skeys[t] = order_key(sc);
      }
    }
    __syncthreads();
  }
  // Not fused: the keys are copied into shared memory once when the launch provided room for them (s_out is unused
  // in this mode and doubles as that flag), so the radix passes do not go back to L2.
  const bool staged = FUSED || s_out != nullptr;
  // the range of the keys, taken along the way: the radix select only has to resolve the bits in which they differ
  uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
  if (!FUSED && staged) {
#pragma unroll 8
    for (int32_t j = tid; j < nr; j += kSelThreads) {  // loads of a trip in flight together
      const uint32_t key = order_key(__ldg(seg + j));
      skeys[j] = key;
      kmin = min(kmin, key);
      kmax = max(kmax, key);
    }
  }
  auto key_at = [&](int32_t j) -> uint32_t { return staged ? skeys[j] : order_key(__ldg(seg + j)); };
  const int32_t lane = tid & 31, warp = tid >> 5;
  if (h > 0) {

  if (FUSED || !staged) {
#pragma unroll 4
    for (int32_t j = tid; j < nr; j += kSelThreads) {
      const uint32_t key = key_at(j);
      kmin = min(kmin, key);
      kmax = max(kmax, key);
    }
  }
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, d));
    kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, d));
  }
  if (lane == 0) { warp_gt[warp] = (int32_t)kmin; warp_eq[warp] = (int32_t)kmax; }
  __syncthreads();
  if (warp == 0) {
    uint32_t a = lane < kSelThreads / 32 ? (uint32_t)warp_gt[lane] : 0xFFFFFFFFu;
    uint32_t b = lane < kSelThreads / 32 ? (uint32_t)warp_eq[lane] : 0u;
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
      a = min(a, __shfl_xor_sync(0xffffffffu, a, d));
      b = max(b, __shfl_xor_sync(0xffffffffu, b, d));
    }
    if (lane == 0) { sh_prefix = a; sh_need = (int32_t)b; }
  }
  __syncthreads();
  kmin = sh_prefix;
  kmax = (uint32_t)sh_need;
  if (tid < 256) hist[tid] = 0;
  __syncthreads();  // sh_prefix / sh_need and the two warp arrays are reused below

  // ---- radix select: the h-th largest key --------------------------------------------
  // MSB first over the bits below the keys' common prefix, 8 at a time (scores of one segment share their sign and
  // most of their exponent: starting at bit 31 would throw nearly every key into one or two bins of the first pass,
  // which the shared-memory atomics would serialise).  The search ends early when the bin that holds the h-th largest
  // key is taken whole: every key of that bin and above is then selected and nothing has to be told apart inside it.
  uint32_t thr;      // keys above thr are selected ...
  int32_t need_eq;   // ... and this many keys equal to thr, lowest positions first
  const uint32_t diff = kmin ^ kmax;
  if (diff == 0u) {
    thr = kmax;
    need_eq = h;
  } else {
    const int32_t nbits = 32 - __clz(diff);  // the keys agree above bit nbits - 1
    uint32_t mask = nbits == 32 ? 0u : ~((1u << nbits) - 1u);
    uint32_t prefix = kmax & mask;
    int32_t need = h;  // rank still to find among keys matching the prefix
    // two block barriers per pass: the warp that reads the bins also clears them for the next pass, and what it
    // publishes is read by everybody before anybody can reach the next pass's first barrier
    for (int32_t shift = max(nbits - 8, 0);; shift = max(shift - 8, 0)) {
#pragma unroll 4
      for (int32_t j = tid; j < nr; j += kSelThreads) {
        const uint32_t key = key_at(j);
        if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
      }
      __syncthreads();
      if (tid < 32) {
        // which bin holds the need-th largest key: bins taken from the top, 8 per lane, a warp scan over the lane sums
        int32_t cnt[8], lane_sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          cnt[i] = hist[255 - 8 * tid - i];
          hist[255 - 8 * tid - i] = 0;
          lane_sum += cnt[i];
        }
        int32_t inc = lane_sum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int32_t x = __shfl_up_sync(0xffffffffu, inc, d);
          if (tid >= d) inc += x;
        }
        int32_t acc = inc - lane_sum;  // keys in the bins above this lane's
        if (acc < need && need <= inc) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if (acc + cnt[i] >= need) {
              // (a digit that overlaps bits already resolved repeats them: or-ing it in changes nothing)
              sh_prefix = prefix | ((uint32_t)(255 - 8 * tid - i) << shift);
              sh_need = need - acc;
              carry_eq = cnt[i];  // size of the chosen bin
              break;
            }
            acc += cnt[i];
          }
        }
      }
      __syncthreads();
      prefix = sh_prefix;
      need = sh_need;
      const int32_t bin = carry_eq;
      mask |= 255u << shift;
      if (bin == need && prefix != 0u) {  // the whole bin: everything at or above its lowest possible key
        thr = prefix - 1u;
        need_eq = 0;
        break;
      }
      if (shift == 0) {
        thr = prefix;  // key of the h-th largest score
        need_eq = need;
        break;
      }
    }
  }

  // ---- ordered compaction: one contiguous run of keys per thread, one block scan ---------------------------------
  // runs of a multiple of 4 keys (128-bit loads) whose number of 16-byte words is odd, so that the quarter-warps'
  // loads fall into different banks
  const int32_t per = 4 * (((nr + kSelThreads * 4 - 1) / (kSelThreads * 4)) | 1);
  const int32_t j0 = min(nr, tid * per), j1 = min(nr, j0 + per);
  int32_t n_gt = 0, n_eq = 0;
  for (int32_t j = j0; j < j1; j += 4) {
    uint32_t k4[4];
    if (staged && j + 4 <= j1) {
      const uint4 q = *reinterpret_cast<const uint4*>(skeys + j);
      k4[0] = q.x; k4[1] = q.y; k4[2] = q.z; k4[3] = q.w;
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) k4[i] = j + i < j1 ? key_at(j + i) : 0u;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const bool valid = j + i < j1;
      n_gt += (valid && k4[i] > thr);
      n_eq += (valid && k4[i] == thr);
    }
  }
  int32_t inc_gt = n_gt, inc_eq = n_eq;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int32_t a = __shfl_up_sync(0xffffffffu, inc_gt, d), b = __shfl_up_sync(0xffffffffu, inc_eq, d);
    if (lane >= d) { inc_gt += a; inc_eq += b; }
  }
  if (lane == 31) { warp_gt[warp] = inc_gt; warp_eq[warp] = inc_eq; }
  __syncthreads();
  if (warp == 0) {
    int32_t a = lane < kSelThreads / 32 ? warp_gt[lane] : 0, b = lane < kSelThreads / 32 ? warp_eq[lane] : 0;
    const int32_t ta = a, tb = b;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int32_t x = __shfl_up_sync(0xffffffffu, a, d), y = __shfl_up_sync(0xffffffffu, b, d);
      if (lane >= d) { a += x; b += y; }
    }
    warp_gt[lane] = a - ta;  // exclusive
    warp_eq[lane] = b - tb;
  }
  __syncthreads();
  int32_t pos_gt = warp_gt[warp] + inc_gt - n_gt;  // exclusive counts before this thread's run
  int32_t pos_eq = warp_eq[warp] + inc_eq - n_eq;
  if (n_gt > 0 || (n_eq > 0 && pos_eq < need_eq)) {
    for (int32_t j = j0; j < j1; ++j) {
      const uint32_t key = key_at(j);
      if (key > thr) {
        out[pos_gt + min(pos_eq, need_eq)] = j;
        ++pos_gt;
      } else if (key == thr) {
        if (pos_eq < need_eq) out[pos_gt + pos_eq] = j;
        ++pos_eq;
      }
    }
  }
  }  // h > 0

  // ---- gather (optional): the CTA copies the rows it has just chosen, K and V, into the compact cache ----------
  if constexpr (GATHER) {
    __syncthreads();  // every index of the segment (written above by this CTA's threads) is visible to all of them
    const int32_t n_keep = h + w, cpr = ga.cpr, rows_per_step = kSelThreads / cpr;
    const int32_t ch = tid % cpr, r_in = tid / cpr;
    const uint4* ks = ga.k_src + layer * ga.src_layer_stride_c;
    const uint4* vs = ga.v_src + layer * ga.src_layer_stride_c;
    uint4* kd = ga.k_dst + layer * ga.dst_layer_stride_c;
    uint4* vd = ga.v_dst + layer * ga.dst_layer_stride_c;
    const int32_t dst0 = cu_kept[r];
    if (r_in < rows_per_step) {
      // four rows of K and of V per thread in flight
      constexpr int kU = 4;
      for (int32_t t0 = r_in; t0 < n_keep; t0 += kU * rows_per_step) {
        uint4 kk[kU], vv[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
          const int32_t t = t0 + u * rows_per_step;
          if (t < n_keep) {
            const int64_t src = ((int64_t)(base + out[t]) * n_kv_heads + g) * cpr + ch;
            kk[u] = ks[src];
            vv[u] = vs[src];
          }
        }
#pragma unroll
        for (int u = 0; u < kU; ++u) {
          const int32_t t = t0 + u * rows_per_step;
          if (t < n_keep) {
            const int64_t dst = ((int64_t)(dst0 + t) * n_kv_heads + g) * cpr + ch;
            kd[dst] = kk[u];
            vd[dst] = vv[u];
          }
        }
      }
    }
  }
}

// Attention sinks + recent window: one CTA per (request, KV head, layer) writes 0 .. h-1 and l-w .. l-1.
__global__ void __launch_bounds__(256) sink_recent_kernel(const int32_t* __restrict__ cu_seqlens,
                                                          const int32_t* __restrict__ cu_kept,
                                                          const int32_t* __restrict__ keep, int32_t window, int32_t k_tot,
                                                          int32_t n_kv_heads, int32_t* __restrict__ idx_out) {
  const int32_t r = blockIdx.x, g = blockIdx.y, layer = blockIdx.z;
  const int32_t len = cu_seqlens[r + 1] - cu_seqlens[r];
  const int32_t w = min(window, len), h = keep[r];
  int32_t* out = idx_out + ((int64_t)layer * n_kv_heads + g) * k_tot + cu_kept[r];
  for (int32_t t = threadIdx.x; t < h + w; t += 256) out[t] = t < h ? t : len - w + (t - h);
}

}  // namespace purekv

using namespace purekv;

extern "C" purekv_status purekv_select_sink_recent(const purekv_batch* batch, int32_t window, const int32_t* keep,
                                                   const int32_t* h_keep, const int32_t* cu_kept, const int32_t* h_cu_kept,
                                                   int32_t n_layers, int32_t n_kv_heads, int32_t* idx_out, void* stream) {
  purekv_status st = check_batch(batch, true);
  if (st != PUREKV_OK) return st;
  if (batch->total_tokens == 0 || batch->n_req == 0 || n_layers == 0) return PUREKV_OK;
  PK_REQUIRE(keep && h_keep && cu_kept && h_cu_kept && idx_out, PUREKV_ERR_INVALID_ARG, "purekv_select_sink_recent: null pointer");
  PK_REQUIRE(n_layers >= 0 && n_layers <= 65535 && n_kv_heads >= 1 && n_kv_heads <= 65535 && window >= 0,
             PUREKV_ERR_INVALID_ARG, "purekv_select_sink_recent: bad sizes");
  PK_REQUIRE(h_cu_kept[0] == 0, PUREKV_ERR_INVALID_ARG, "cu_kept[0] must be 0");
  for (int r = 0; r < batch->n_req; ++r) {
    const int32_t len = batch->h_cu_seqlens[r + 1] - batch->h_cu_seqlens[r];
    const int32_t w = std::min(window, len);
    PK_REQUIRE(h_keep[r] >= 0 && h_keep[r] <= len - w && h_cu_kept[r + 1] - h_cu_kept[r] == h_keep[r] + w,
               PUREKV_ERR_INVALID_ARG, "request %d: h = %d must lie in [0, %d] and its kept count be h + w", r, h_keep[r],
               len - w);
  }
  dim3 grid((unsigned)batch->n_req, (unsigned)n_kv_heads, (unsigned)n_layers);
  sink_recent_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(batch->cu_seqlens, cu_kept, keep, window,
                                                             h_cu_kept[batch->n_req], n_kv_heads, idx_out);
  PK_CUDA(cudaGetLastError());
  return PUREKV_OK;
}

extern "C" size_t purekv_select_ws_bytes(const purekv_batch* batch, int32_t n_layers, int32_t n_kv_heads) {
  if (!batch || n_layers < 0 || n_kv_heads < 0) return 0;
  return (size_t)n_layers * n_kv_heads * batch->total_tokens * sizeof(float) + 256;
}

// Common body of purekv_select_topk and purekv_select_compact (ga.k_src != nullptr: the selecting CTAs also gather).
static purekv_status select_impl(const float* c, const void* v, int64_t v_layer_stride, int32_t n_layers,
                                 const purekv_batch* batch, int32_t window, const int32_t* keep, const int32_t* h_keep,
                                 const int32_t* cu_kept, const int32_t* h_cu_kept, int32_t n_kv_heads, int32_t head_dim,
                                 purekv_dtype dtype, int32_t* idx_out, float* s_out, void* ws, size_t ws_bytes,
                                 void* stream, Gather ga) {
  purekv_status st = check_batch(batch, true);
  if (st != PUREKV_OK) return st;
  if (batch->total_tokens == 0 || batch->n_req == 0) return PUREKV_OK;  // empty batch: nothing to do
  PK_REQUIRE(c && v && keep && h_keep && cu_kept && h_cu_kept && idx_out, PUREKV_ERR_INVALID_ARG,
             "purekv_select_topk: null pointer");
  PK_REQUIRE(n_layers >= 0 && n_layers <= 65535 && n_kv_heads >= 1 && n_kv_heads <= 65535 && head_dim >= 1 &&
                 window >= 0,
             PUREKV_ERR_INVALID_ARG, "purekv_select_topk: bad sizes");
  PK_REQUIRE(dtype == PUREKV_BF16 || dtype == PUREKV_FP32, PUREKV_ERR_INVALID_ARG, "unknown dtype");
  const int64_t esz = dtype == PUREKV_BF16 ? 2 : 4;
  PK_REQUIRE((head_dim * esz) % 16 == 0, PUREKV_ERR_UNSUPPORTED, "V row of %lld bytes is not a multiple of 16",
             (long long)(head_dim * esz));
  PK_REQUIRE((v_layer_stride * esz) % 16 == 0 && (uintptr_t)v % 16 == 0, PUREKV_ERR_INVALID_ARG,
             "V base and layer stride must be 16-byte aligned");
  PK_REQUIRE(h_cu_kept[0] == 0, PUREKV_ERR_INVALID_ARG, "cu_kept[0] must be 0");
  for (int r = 0; r < batch->n_req; ++r) {
    const int32_t len = batch->h_cu_seqlens[r + 1] - batch->h_cu_seqlens[r];
    const int32_t w = std::min(window, len);
    PK_REQUIRE(h_keep[r] >= 0 && h_keep[r] <= len - w, PUREKV_ERR_INVALID_ARG,
               "request %d: h = %d outside [0, %d]", r, h_keep[r], len - w);
    PK_REQUIRE(h_cu_kept[r + 1] - h_cu_kept[r] == h_keep[r] + w, PUREKV_ERR_INVALID_ARG,
               "request %d: cu_kept step %d != h + w = %d", r, h_cu_kept[r + 1] - h_cu_kept[r], h_keep[r] + w);
  }
  const int64_t T = batch->total_tokens;
  if (n_layers == 0 || T == 0 || batch->n_req == 0) return PUREKV_OK;
  cudaStream_t sm = (cudaStream_t)stream;
  const int32_t cpr = (int32_t)(head_dim * esz / 16);
  dim3 g2((unsigned)batch->n_req, (unsigned)n_kv_heads, (unsigned)n_layers);
  const int32_t k_tot = h_cu_kept[batch->n_req];
  // Fused path: each (request, head, layer) segment is streamed, scored and selected by one CTA.  It needs 256-byte
  // rows, the segment's keys in shared memory, and enough segments to occupy the SMs; otherwise V is streamed by a
  // grid-wide kernel first and the selection reads the scores back.
  int32_t longest = 0;
  for (int r = 0; r < batch->n_req; ++r) longest = std::max(longest, batch->h_cu_seqlens[r + 1] - batch->h_cu_seqlens[r]);
  const size_t key_bytes = (size_t)longest * sizeof(uint32_t);
  const int64_t segments = (int64_t)batch->n_req * n_kv_heads * n_layers;
  if (cpr == 16 && key_bytes <= 200 * 1024 && segments >= 2 * 148) {
    auto launch_fused = [&](auto kernel, std::atomic<uint64_t>& smem_allowed) -> purekv_status {
      const purekv_status st_smem = allow_max_dynamic_smem(kernel, smem_allowed);
      if (st_smem != PUREKV_OK) return st_smem;
      kernel<<<g2, kSelThreads, key_bytes, sm>>>(nullptr, T, batch->cu_seqlens, cu_kept, keep, window, k_tot, n_kv_heads,
                                                 idx_out, (const uint4*)v, v_layer_stride * esz / 16, c, s_out, ga);
      PK_CUDA(cudaGetLastError());
      return PUREKV_OK;
    };
    static std::atomic<uint64_t> allowed[4] = {{0}, {0}, {0}, {0}};
    const bool gather = ga.k_src != nullptr;
    if (dtype == PUREKV_BF16)
      return gather ? launch_fused(select_kernel<true, __nv_bfloat16, true>, allowed[0])
                    : launch_fused(select_kernel<true, __nv_bfloat16, false>, allowed[1]);
    return gather ? launch_fused(select_kernel<true, float, true>, allowed[2])
                  : launch_fused(select_kernel<true, float, false>, allowed[3]);
  }
  float* s_buf = s_out;
  if (!s_buf) {
    PK_REQUIRE(ws && ws_bytes >= purekv_select_ws_bytes(batch, n_layers, n_kv_heads), PUREKV_ERR_WORKSPACE,
               "purekv_select_topk: workspace of %zu bytes is too small", ws_bytes);
    s_buf = (float*)(((uintptr_t)ws + 255) & ~(uintptr_t)255);
  }
  const int64_t n_items = ((T * n_kv_heads + 31) / 32) * n_layers;  // blocks of 32 (token, head) rows per layer
  dim3 g1((unsigned)std::min<int64_t>((n_items + 7) / 8, 148 * 3));   // one wave: 3 CTAs of 256 threads per SM (measured best)
  if (dtype == PUREKV_BF16)
    vnorm_score_kernel<__nv_bfloat16><<<g1, 256, 0, sm>>>((const uint4*)v, v_layer_stride * esz / 16, c, T, n_kv_heads,
                                                          n_layers, cpr, s_buf);
  else
    vnorm_score_kernel<float><<<g1, 256, 0, sm>>>((const uint4*)v, v_layer_stride * esz / 16, c, T, n_kv_heads, n_layers,
                                                  cpr, s_buf);
  PK_CUDA(cudaGetLastError());
  const bool stage_keys = key_bytes <= 200 * 1024;
  const bool gather = ga.k_src != nullptr;
  if (stage_keys) {
    static std::atomic<uint64_t> smem_allowed{0}, smem_allowed_g{0};
    const purekv_status st_smem = gather ? allow_max_dynamic_smem(select_kernel<false, float, true>, smem_allowed_g)
                                         : allow_max_dynamic_smem(select_kernel<false, float, false>, smem_allowed);
    if (st_smem != PUREKV_OK) return st_smem;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = g2;
  cfg.blockDim = dim3(kSelThreads);
  cfg.dynamicSmemBytes = stage_keys ? key_bytes : 0;
  cfg.stream = sm;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see griddepcontrol in the two kernels
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (gather)
    PK_CUDA(cudaLaunchKernelEx(&cfg, select_kernel<false, float, true>, (const float*)s_buf, T, batch->cu_seqlens, cu_kept,
                               keep, window, k_tot, n_kv_heads, idx_out, (const uint4*)nullptr, (int64_t)0,
                               (const float*)nullptr, stage_keys ? s_buf : (float*)nullptr, ga));
  else
    PK_CUDA(cudaLaunchKernelEx(&cfg, select_kernel<false, float, false>, (const float*)s_buf, T, batch->cu_seqlens, cu_kept,
                               keep, window, k_tot, n_kv_heads, idx_out, (const uint4*)nullptr, (int64_t)0,
                               (const float*)nullptr, stage_keys ? s_buf : (float*)nullptr, ga));
  PK_CUDA(cudaGetLastError());
  return PUREKV_OK;
}

extern "C" purekv_status purekv_select_topk(const float* c, const void* v, int64_t v_layer_stride, int32_t n_layers,
                                            const purekv_batch* batch, int32_t window, const int32_t* keep,
                                            const int32_t* h_keep, const int32_t* cu_kept, const int32_t* h_cu_kept,
                                            int32_t n_kv_heads, int32_t head_dim, purekv_dtype dtype,
                                            int32_t* idx_out, float* s_out, void* ws, size_t ws_bytes, void* stream) {
  return select_impl(c, v, v_layer_stride, n_layers, batch, window, keep, h_keep, cu_kept, h_cu_kept, n_kv_heads, head_dim,
                     dtype, idx_out, s_out, ws, ws_bytes, stream, Gather{});
}

extern "C" purekv_status purekv_select_compact(const float* c, const void* k, const void* v, int64_t layer_stride,
                                               int32_t n_layers, const purekv_batch* batch, int32_t window,
                                               const int32_t* keep, const int32_t* h_keep, const int32_t* cu_kept,
                                               const int32_t* h_cu_kept, int32_t n_kv_heads, int32_t head_dim,
                                               purekv_dtype dtype, int32_t* idx_out, float* s_out, void* k_out,
                                               void* v_out, int64_t out_layer_stride, void* ws, size_t ws_bytes,
                                               void* stream) {
  PK_REQUIRE(k && k_out && v_out, PUREKV_ERR_INVALID_ARG, "purekv_select_compact: null pointer");
  PK_REQUIRE(dtype == PUREKV_BF16 || dtype == PUREKV_FP32, PUREKV_ERR_INVALID_ARG, "unknown dtype");
  const int64_t esz = dtype == PUREKV_BF16 ? 2 : 4;
  PK_REQUIRE(head_dim >= 1 && (head_dim * esz) % 16 == 0 && head_dim * esz / 16 <= kSelThreads, PUREKV_ERR_UNSUPPORTED,
             "row of %lld bytes: need a multiple of 16 up to %d", (long long)(head_dim * esz), 16 * kSelThreads);
  PK_REQUIRE((layer_stride * esz) % 16 == 0 && (out_layer_stride * esz) % 16 == 0 &&
                 ((uintptr_t)k | (uintptr_t)v | (uintptr_t)k_out | (uintptr_t)v_out) % 16 == 0,
             PUREKV_ERR_INVALID_ARG, "K/V bases and layer strides must be 16-byte aligned");
  Gather ga;
  ga.k_src = (const uint4*)k;
  ga.v_src = (const uint4*)v;
  ga.k_dst = (uint4*)k_out;
  ga.v_dst = (uint4*)v_out;
  ga.src_layer_stride_c = layer_stride * esz / 16;
  ga.dst_layer_stride_c = out_layer_stride * esz / 16;
  ga.cpr = (int32_t)(head_dim * esz / 16);
  return select_impl(c, v, layer_stride, n_layers, batch, window, keep, h_keep, cu_kept, h_cu_kept, n_kv_heads, head_dim,
                     dtype, idx_out, s_out, ws, ws_bytes, stream, ga);
}
