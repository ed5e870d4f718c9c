// purekv_lowlayer_score_lse: window column sums (Eq. 2) on the tcgen05 tensor cores, given the rows' log-sum-exp.
//
// When the scored layer's dense causal prefill has already produced the log-sum-exp of every row (Eq. 1's row
// normaliser), the scores need one pass: C[g, j] = (1/G) sum over the G*w stacked window rows of exp(s - lse).
// An item is 128 keys of one (request, KV head) -- one key per TMEM lane --; a CTA walks its stacked rows in blocks
// of 128 columns: S^T = K Q_w^T with tcgen05.mma (A = the K tile, B = a block of window rows, both K-major from
// shared memory, fp32 accumulators in TMEM, two buffers).  Roles:
//   warp 0      producer: the K tile once, then per block of rows 128 / B boxes of B rows per 64-column panel, B the
//               largest power of two (at most 128) that divides every request's window: a block of stacked rows
//               may span several query heads, a box of B rows never does (few large boxes: the copy engine's rate
//               of small boxes bounded this kernel when the boxes were 8 rows high)
//   warp 1      owns the TMEM columns; one lane issues the products
//   warps 2-9   two groups of four warps, one thread per key in each; a group takes every other block of rows (always
//               the same accumulator): S^T row from TMEM, exp2 against the column's log-sum-exp, running sum; the
//               groups' sums meet at the end.  Two CTAs per SM give each scheduler four such warps: with two the
//               kernel was bound by the latencies of the TMEM loads and of the exponentials, not by any unit's rate.
// Two launch forms share these roles: one CTA per item (score_tc_kernel) for long lists of rows, and two persistent
// CTAs per SM that take the items in turn (score_tc_items_kernel) for short ones, where barriers, TMEM and the
// pipeline's phases carry over from item to item and an item's loads overlap the previous item's sums.
// bf16, head_dim 128, window a multiple of 8.  Every wait is bounded; on expiry the status word is set.
#include <algorithm>

#include "tc_util.cuh"

namespace purekv {
namespace sc {

// Of the eight groups of four logits in a 32-column chunk, this many take the second pair's exponentials as a cubic
// on the FMA pipe instead of the MUFU unit (relative error 7.5e-5 against a score tolerance of 1e-3).
#ifndef PUREKV_SCORE_POLY
#define PUREKV_SCORE_POLY 6
#endif
constexpr int kScorePoly = PUREKV_SCORE_POLY;
using namespace tc;

constexpr int kKeys = 128, kRows = 128;
constexpr int kThreads = 320;
constexpr int kStages = 2;         // Q-row blocks in flight
constexpr uint32_t kTmemCols = 256;  // two 128-column accumulators
constexpr uint32_t kPanel = kRows * 128;  // bytes of one 64-column panel of a 128-row tile
constexpr uint32_t kTile = 2 * kPanel;

struct __align__(8) Barriers {
  uint64_t k_full;
  uint64_t q_full[kStages], q_empty[kStages];
  uint64_t d_full[2], d_empty[2];
  uint64_t drain;
};

// One CTA per key block of a (request, KV head), handed out by the hardware: the form used when an item's list of
// rows is long (see the launch code).
__global__ void __launch_bounds__(kThreads, 2) score_tc_kernel(
    const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q8, const float* __restrict__ lse,
    float* __restrict__ c_out, const int32_t* __restrict__ cu_seqlens, int32_t window, int32_t n_q_heads,
    int32_t n_kv_heads, float scale_log2, int64_t n_tokens, int32_t* __restrict__ status, uint64_t wait_ns,
    int32_t box_rows) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ Barriers bars;
  __shared__ __align__(16) float lse_s[8][2][kRows];  // per epilogue warp: the log-sum-exp values of two blocks of rows
  __shared__ float comb_s[kKeys];                     // the second group's column sums, for the first to add
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  const int32_t r = blockIdx.z, g = blockIdx.y, j0 = blockIdx.x * kKeys;
  const int32_t G = n_q_heads / n_kv_heads;
  const int32_t base = cu_seqlens[r], len = cu_seqlens[r + 1] - base;
  const int32_t w = min(window, len), nr = len - w, n_rows = G * w;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (j0 >= len) return;
  float* cg = c_out + (int64_t)g * n_tokens + base;
  if (j0 >= nr) {  // block inside the window: defined as 0 (before any barrier or TMEM work)
    for (int c = tid; c < kKeys; c += kThreads)
      if (j0 + c < len) cg[j0 + c] = 0.f;
    return;
  }
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sK = smem0;          // [2 panels][128 keys x 128 B]
  const uint32_t sQ = sK + kTile;     // [kStages][2 panels][128 rows x 128 B]
  const int32_t n_blocks = (n_rows + kRows - 1) / kRows;
  // Every CTA of a (request, KV head) reads the same blocks of window rows, and CTAs of one wave run in step: started
  // at the same block they would all pull the same lines from the same L2 slices at the same time.  Each CTA
  // therefore starts its walk at a different block (the column sums do not depend on the order).
  const int32_t rot = (int32_t)(blockIdx.x % (uint32_t)n_blocks);
  volatile int* abort_flag = &abort_s;

  if (tid == 0) {
    abort_s = *reinterpret_cast<volatile int32_t*>(status) != 0;
    mbar_init(smem_u32(&bars.k_full), 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&bars.q_full[s]), 1);
      mbar_init(smem_u32(&bars.q_empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars.d_full[b]), 1);
      mbar_init(smem_u32(&bars.d_empty[b]), 4);  // one arrival per epilogue warp
    }
    mbar_init(smem_u32(&bars.drain), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_s), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  const bool start_ok = abort_s == 0;
  float col_sum = 0.f;  // an epilogue thread's column sum over its group's blocks

  if (start_ok && warp == 0) {
    // ---------------- producer ----------------
    if (lane == 0) {
      mbar_expect_tx(smem_u32(&bars.k_full), kTile);
      tma_load_3d(sK, &tm_k, smem_u32(&bars.k_full), 0, g, base + j0);
      tma_load_3d(sK + kPanel, &tm_k, smem_u32(&bars.k_full), 64, g, base + j0);
      int32_t issued = 0;
      for (int32_t t = 0; t < n_blocks; ++t) {
        const int32_t s = t % kStages;
        if (t >= kStages && !mbar_wait(smem_u32(&bars.q_empty[s]), ((t / kStages) - 1) & 1, abort_flag, wait_ns)) break;
        mbar_expect_tx(smem_u32(&bars.q_full[s]), kTile);
        for (int32_t grp = 0; grp < kRows / box_rows; ++grp) {
          const int32_t row = ((t + rot) % n_blocks) * kRows + box_rows * grp;
          // rows past the stacked list read from beyond the tensor: zero fill
          int32_t tok = (int32_t)n_tokens, head = 0;
          if (row < n_rows) {
            tok = base + len - w + row % w;
            head = g * G + row / w;
          }
          const uint32_t dst = sQ + s * kTile + grp * (box_rows * 128);
          tma_load_3d(dst, &tm_q8, smem_u32(&bars.q_full[s]), 0, head, tok);
          tma_load_3d(dst + kPanel, &tm_q8, smem_u32(&bars.q_full[s]), 64, head, tok);
        }
        issued = t + 1;
      }
      if (*abort_flag) {  // every issued copy must have landed before shared memory is released
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(smem_u32(&bars.k_full), 0) && global_ns() - t0 < wait_ns) {}
        for (int32_t t = max(0, issued - kStages); t < issued; ++t)
          while (!mbar_try_wait(smem_u32(&bars.q_full[t % kStages]), (t / kStages) & 1) && global_ns() - t0 < wait_ns) {}
      }
    }
  } else if (start_ok && warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(kRows, false);
      constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
      const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
      const uint32_t q_lo0 = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
      bool ok = mbar_wait(smem_u32(&bars.k_full), 0, abort_flag, wait_ns);
      for (int32_t t = 0; ok && t < n_blocks; ++t) {
        const int32_t s = t % kStages, b = t & 1;
        ok = mbar_wait(smem_u32(&bars.q_full[s]), (t / kStages) & 1, abort_flag, wait_ns);
        if (ok && t >= 2) ok = mbar_wait(smem_u32(&bars.d_empty[b]), ((t >> 1) - 1) & 1, abort_flag, wait_ns);
        if (!ok) break;
        tc_fence_after();
        const uint32_t q_lo = q_lo0 + s * (kTile >> 4);
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks)
          mma_ss_lh(tmem + b * kRows, k_lo0 + (ks >> 2) * (kPanel >> 4) + (ks & 3) * 2, kDescHi,
                    q_lo + (ks >> 2) * (kPanel >> 4) + (ks & 3) * 2, kDescHi, idesc, ks > 0 ? 1u : 0u);
        tc_commit(smem_u32(&bars.d_full[b]));
        tc_commit(smem_u32(&bars.q_empty[s]));
      }
      if (!ok) {  // leaving early: let every issued MMA finish before TMEM is released
        tc_commit(smem_u32(&bars.drain));
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(smem_u32(&bars.drain), 0) && global_ns() - t0 < wait_ns) {}
      }
    }
  } else if (start_ok && warp >= 2) {
    // ---------------- column sums: one thread per key ----------------
    const int quad = warp & 3;  // TMEM lane quadrant this warp may access
    const int32_t wg = (warp - 2) >> 2;  // this warp's group takes blocks wg, wg + 2, ...: always accumulator wg
    const int key = quad * 32 + lane;
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16);
    const float kLog2e = 1.4426950408889634f;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    bool ok = true;
    // The log-sum-exp of a block's 128 stacked rows (log2 units; +inf for absent rows): every key needs all of them.
    // Each warp keeps its own copy in shared memory, fetched one block ahead (lane i loads rows i, i+32, i+64, i+96)
    // and read back four at a time; no meeting between warps is needed.
    float (*my_lse)[kRows] = lse_s[warp - 2];
    const uint32_t w_inv = (uint32_t)(0x100000000ull / (uint32_t)w);  // floor(2^32 / w): the quotient estimate is low by at most 1
    auto fetch_lse = [&](int32_t t, float (&lv)[4]) {
      const int32_t blk = t + rot < n_blocks ? t + rot : t + rot - n_blocks;  // t and rot are both below n_blocks
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int32_t row = blk * kRows + 32 * c + lane;
        lv[c] = INFINITY;
        if (row < n_rows) {
          // row / w by a multiplication (a division per row and block is a tenth of this warp's instructions)
          int32_t head = (int32_t)__umulhi((uint32_t)row, w_inv);
          head += (head + 1) * w <= row;
          lv[c] = __ldg(lse + (int64_t)(g * G + head) * n_tokens + base + len - w + (row - head * w)) * kLog2e;
        }
      }
    };
    float lv[4];
    if (wg < n_blocks) {
      fetch_lse(wg, lv);
#pragma unroll
      for (int c = 0; c < 4; ++c) my_lse[0][32 * c + lane] = lv[c];
    }
    __syncwarp();
    for (int32_t t = wg, n = 0; ok && t < n_blocks; t += 2, ++n) {
      const int32_t b = wg, lb = n & 1;
      if (t + 2 < n_blocks) fetch_lse(t + 2, lv);  // in flight while this block is summed
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.d_full[b]), (t >> 1) & 1, abort_flag, wait_ns) ? 1 : 0) != 0;
      if (!ok) break;
      tc_fence_after();
      const float4* l4 = reinterpret_cast<const float4*>(my_lse[lb]);
      // the next 32 columns are on their way from TMEM while the current ones go through the exponentials
      uint32_t rr[2][32];
      tmem_ld32(t_lane + b * kRows, rr[0]);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        tc_wait_ld();
        if (c + 1 < 4) tmem_ld32(t_lane + b * kRows + 32 * (c + 1), rr[(c + 1) & 1]);
#pragma unroll
        for (int x = 0; x < 32; x += 4) {
          const float4 l = l4[8 * c + (x >> 2)];
          acc[0] += ex2(fmaf(__uint_as_float(rr[c & 1][x]), scale_log2, -l.x));
          acc[1] += ex2(fmaf(__uint_as_float(rr[c & 1][x + 1]), scale_log2, -l.y));
          if ((x >> 2) < kScorePoly) {
            // this pair's exponentials on the FMA pipe: the kernel is paced by the MUFU unit (one ex2 per logit)
            const float2 a = __ffma2_rn(make_float2(__uint_as_float(rr[c & 1][x + 2]), __uint_as_float(rr[c & 1][x + 3])),
                                        make_float2(scale_log2, scale_log2), make_float2(-l.z, -l.w));
            const float2 pp = exp2_poly2(a);
            acc[2] += pp.x;
            acc[3] += pp.y;
          } else {
            acc[2] += ex2(fmaf(__uint_as_float(rr[c & 1][x + 2]), scale_log2, -l.z));
            acc[3] += ex2(fmaf(__uint_as_float(rr[c & 1][x + 3]), scale_log2, -l.w));
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars.d_empty[b]));
      if (t + 2 < n_blocks) {
#pragma unroll
        for (int c = 0; c < 4; ++c) my_lse[lb ^ 1][32 * c + lane] = lv[c];  // last read two of this warp's blocks ago
        __syncwarp();
      }
    }
    // the two groups' sums meet after the CTA's closing barrier
    col_sum = (acc[0] + acc[1]) + (acc[2] + acc[3]);
    if (wg == 1) comb_s[key] = col_sum;
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
  if (start_ok && warp >= 2 && warp < 6 && abort_s == 0) {
    const int32_t j = j0 + (warp & 3) * 32 + lane;
    if (j < len) cg[j] = j < nr ? (col_sum + comb_s[(warp & 3) * 32 + lane]) / (float)G : 0.f;
  }
  if (tid == 0 && abort_s && start_ok) atomicExch(status, (int32_t)PUREKV_ERR_TIMEOUT);
}


// ---- the persistent form -------------------------------------------------------------------------------------------
struct __align__(8) ItemBarriers {
  uint64_t k_full, k_empty;
  uint64_t q_full[kStages], q_empty[kStages];
  uint64_t d_full[2], d_empty[2];
  uint64_t comb_full, comb_empty;  // the second group's column sums are in comb_s / have been taken from it
  uint64_t drain;
};

// One item: a key block of one (request, KV head).  Items are numbered request by request, head by head, block by
// block over the blocks each request really has; every role decodes an item's number the same way, through the
// running block counts of the requests that the CTA builds in shared memory when it starts.
constexpr int kMaxReq = 1024;  // requests the table holds (larger batches take the one-CTA-per-item form)
struct Item {
  int32_t g, j0;             // KV head, first key of the block
  int32_t base, len, w, nr;  // the request's first token, length, clipped window, keys outside the window
  int32_t n_blocks, rot;     // blocks of 128 stacked window rows; the block this item's walk starts at
  int32_t kind;              // 0: none; 1: inside the window, scores are 0; 2: products
  int32_t number;            // the item's number
  uint32_t w_inv;            // floor(2^32 / w), set by the roles that divide by w often
};

__device__ __forceinline__ Item decode_item(int32_t item, const int32_t* blk_prefix, int32_t n_req, int32_t n_kv_heads,
                                            int32_t G, int32_t window, const int32_t* __restrict__ cu_seqlens) {
  Item it;
  // the request: the last r whose first item is at or before this one (requests without tokens have no items)
  int32_t lo = 0, hi = n_req - 1;
  while (lo < hi) {
    const int32_t mid = (lo + hi + 1) >> 1;
    if (blk_prefix[mid] * n_kv_heads <= item) lo = mid;
    else hi = mid - 1;
  }
  const int32_t r = lo, nb = blk_prefix[r + 1] - blk_prefix[r], rem = item - blk_prefix[r] * n_kv_heads;
  const int32_t x = rem % nb;
  it.g = rem / nb;
  it.j0 = x * kKeys;
  it.base = __ldg(cu_seqlens + r);
  it.len = __ldg(cu_seqlens + r + 1) - it.base;
  it.w = min(window, it.len);
  it.nr = it.len - it.w;
  it.n_blocks = (G * it.w + kRows - 1) / kRows;
  // Every CTA that works on a (request, KV head) reads the same blocks of window rows, and CTAs run in step: started
  // at the same block they would all pull the same lines from the same L2 slices at the same time.  Each key block
  // therefore starts its walk at a different block (the column sums do not depend on the order).
  it.rot = x % it.n_blocks;
  it.kind = it.j0 >= it.nr ? 1 : 2;
  it.number = item;
  it.w_inv = 0u;
  return it;
}

// The grid's CTAs (two per SM) take the items in turn, item = blockIdx.x + k * gridDim.x; barriers, TMEM and the
// pipeline's phases carry over from one item to the next, so that an item's fixed costs (tile loads, first product,
// the rows' log-sum-exp) overlap the previous item's sums.
__global__ void __launch_bounds__(kThreads, 2) score_tc_items_kernel(
    const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q8, const float* __restrict__ lse,
    float* __restrict__ c_out, const int32_t* __restrict__ cu_seqlens, int32_t window, int32_t n_q_heads,
    int32_t n_kv_heads, float scale_log2, int64_t n_tokens, int32_t* __restrict__ status, uint64_t wait_ns,
    int32_t box_rows, int32_t n_req, int32_t n_items) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ ItemBarriers bars;
  __shared__ __align__(16) float lse_s[8][2][kRows];  // per epilogue warp: the log-sum-exp values of two blocks of rows
  __shared__ float comb_s[kKeys];                     // the second group's column sums, for the first to add
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  __shared__ int32_t blk_prefix[kMaxReq + 1];  // key blocks of the requests before each request
  const int32_t G = n_q_heads / n_kv_heads;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sK = smem0;          // [2 panels][128 keys x 128 B]
  const uint32_t sQ = sK + kTile;     // [kStages][2 panels][128 rows x 128 B]
  volatile int* abort_flag = &abort_s;

  // running block counts: every thread counts a few requests, then one warp scans the counts 32 at a time
  for (int32_t r = tid; r < n_req; r += kThreads)
    blk_prefix[r + 1] = (__ldg(cu_seqlens + r + 1) - __ldg(cu_seqlens + r) + kKeys - 1) / kKeys;
  if (tid == 0) blk_prefix[0] = 0;
  __syncthreads();
  if (warp == 0) {
    int32_t carry = 0;
    for (int32_t r0 = 0; r0 < n_req; r0 += 32) {
      int32_t v = r0 + lane < n_req ? blk_prefix[r0 + lane + 1] : 0;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int32_t y = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += y;
      }
      if (r0 + lane < n_req) blk_prefix[r0 + lane + 1] = carry + v;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
  }
  if (tid == 0) {
    abort_s = *reinterpret_cast<volatile int32_t*>(status) != 0;
    mbar_init(smem_u32(&bars.k_full), 1);
    mbar_init(smem_u32(&bars.k_empty), 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&bars.q_full[s]), 1);
      mbar_init(smem_u32(&bars.q_empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars.d_full[b]), 1);
      mbar_init(smem_u32(&bars.d_empty[b]), 4);  // one arrival per epilogue warp of the group that owns the buffer
    }
    mbar_init(smem_u32(&bars.comb_full), 4);
    mbar_init(smem_u32(&bars.comb_empty), 4);
    mbar_init(smem_u32(&bars.drain), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_s), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  const bool start_ok = abort_s == 0;
  const int32_t item0 = (int32_t)blockIdx.x, stride = (int32_t)gridDim.x;

  if (start_ok && warp == 0) {
    // ---------------- producer ----------------
    if (lane == 0) {
      uint32_t u = 0, nc = 0;  // blocks of rows and items with products, so far
      int32_t issued_q = 0, issued_k = 0;
      bool ok = true;
      for (int32_t item = item0; ok && item < n_items; item += stride) {
        const Item it = decode_item(item, blk_prefix, n_req, n_kv_heads, G, window, cu_seqlens);
        if (it.kind != 2) continue;
        if (nc > 0 && !mbar_wait(smem_u32(&bars.k_empty), (nc - 1u) & 1u, abort_flag, wait_ns)) break;
        mbar_expect_tx(smem_u32(&bars.k_full), kTile);
        tma_load_3d(sK, &tm_k, smem_u32(&bars.k_full), 0, it.g, it.base + it.j0);
        tma_load_3d(sK + kPanel, &tm_k, smem_u32(&bars.k_full), 64, it.g, it.base + it.j0);
        issued_k = (int32_t)nc + 1;
        const int32_t n_rows = G * it.w;
        for (int32_t t = 0; t < it.n_blocks; ++t, ++u) {
          const uint32_t s = u % kStages;
          if (u >= (uint32_t)kStages && !mbar_wait(smem_u32(&bars.q_empty[s]), ((u / kStages) - 1u) & 1u, abort_flag, wait_ns)) {
            ok = false;
            break;
          }
          mbar_expect_tx(smem_u32(&bars.q_full[s]), kTile);
          const int32_t blk = t + it.rot < it.n_blocks ? t + it.rot : t + it.rot - it.n_blocks;
          for (int32_t grp = 0; grp < kRows / box_rows; ++grp) {
            const int32_t row = blk * kRows + box_rows * grp;
            // rows past the stacked list read from beyond the tensor: zero fill
            int32_t tok = (int32_t)n_tokens, head = 0;
            if (row < n_rows) {
              tok = it.base + it.len - it.w + row % it.w;
              head = it.g * G + row / it.w;
            }
            const uint32_t dst = sQ + s * kTile + grp * (box_rows * 128);
            tma_load_3d(dst, &tm_q8, smem_u32(&bars.q_full[s]), 0, head, tok);
            tma_load_3d(dst + kPanel, &tm_q8, smem_u32(&bars.q_full[s]), 64, head, tok);
          }
          issued_q = (int32_t)u + 1;
        }
        ++nc;
      }
      if (*abort_flag) {  // every issued copy must have landed before shared memory is released
        const uint64_t t0 = global_ns();
        if (issued_k > 0)
          while (!mbar_try_wait(smem_u32(&bars.k_full), (uint32_t)(issued_k - 1) & 1u) && global_ns() - t0 < wait_ns) {}
        for (int32_t t = max(0, issued_q - kStages); t < issued_q; ++t)
          while (!mbar_try_wait(smem_u32(&bars.q_full[t % kStages]), (t / kStages) & 1) && global_ns() - t0 < wait_ns) {}
      }
    }
  } else if (start_ok && warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(kRows, false);
      constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
      const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
      const uint32_t q_lo0 = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
      uint32_t u = 0, nc = 0;
      bool ok = true;
      for (int32_t item = item0; ok && item < n_items; item += stride) {
        const Item it = decode_item(item, blk_prefix, n_req, n_kv_heads, G, window, cu_seqlens);
        if (it.kind != 2) continue;
        ok = mbar_wait(smem_u32(&bars.k_full), nc & 1u, abort_flag, wait_ns);
        for (int32_t t = 0; ok && t < it.n_blocks; ++t, ++u) {
          const uint32_t s = u % kStages, b = u & 1u;
          ok = mbar_wait(smem_u32(&bars.q_full[s]), (u / kStages) & 1u, abort_flag, wait_ns);
          if (ok && u >= 2u) ok = mbar_wait(smem_u32(&bars.d_empty[b]), ((u >> 1) - 1u) & 1u, abort_flag, wait_ns);
          if (!ok) break;
          tc_fence_after();
          const uint32_t q_lo = q_lo0 + s * (kTile >> 4);
#pragma unroll
          for (int ks = 0; ks < kD / 16; ++ks)
            mma_ss_lh(tmem + b * kRows, k_lo0 + (ks >> 2) * (kPanel >> 4) + (ks & 3) * 2, kDescHi,
                      q_lo + (ks >> 2) * (kPanel >> 4) + (ks & 3) * 2, kDescHi, idesc, ks > 0 ? 1u : 0u);
          tc_commit(smem_u32(&bars.d_full[b]));
          tc_commit(smem_u32(&bars.q_empty[s]));
        }
        if (ok) tc_commit(smem_u32(&bars.k_empty));  // the item's last read of the K tile
        ++nc;
      }
      if (!ok) {  // leaving early: let every issued MMA finish before TMEM is released
        tc_commit(smem_u32(&bars.drain));
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(smem_u32(&bars.drain), 0) && global_ns() - t0 < wait_ns) {}
      }
    }
  } else if (start_ok && warp >= 2) {
    // ---------------- column sums: one thread per key ----------------
    const int quad = warp & 3;  // TMEM lane quadrant this warp may access
    // this warp's group takes the blocks whose running number has parity wg: always accumulator wg
    const uint32_t wg = (uint32_t)(warp - 2) >> 2;
    const int key = quad * 32 + lane;
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16);
    const float kLog2e = 1.4426950408889634f;
    bool ok = true;
    // The log-sum-exp of a block's 128 stacked rows (log2 units; +inf for absent rows): every key needs all of them.
    // Each warp keeps its own copy in shared memory, fetched one block ahead -- across items too -- (lane i loads rows
    // i, i+32, i+64, i+96) and read back four at a time; no meeting between warps is needed.
    float (*my_lse)[kRows] = lse_s[warp - 2];
    auto fetch_lse = [&](const Item& it, int32_t t, float (&lv)[4]) {
      const int32_t blk = t + it.rot < it.n_blocks ? t + it.rot : t + it.rot - it.n_blocks;  // t and rot are both below n_blocks
      const int32_t n_rows = G * it.w;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int32_t row = blk * kRows + 32 * c + lane;
        lv[c] = INFINITY;
        if (row < n_rows) {
          // row / w by a multiplication; the estimate from floor(2^32 / w) is low by at most 1
          int32_t head = (int32_t)__umulhi((uint32_t)row, it.w_inv);
          head += (head + 1) * it.w <= row;
          lv[c] = __ldg(lse + (int64_t)(it.g * G + head) * n_tokens + it.base + it.len - it.w + (row - head * it.w)) * kLog2e;
        }
      }
    };
    // the next item with products from `item` on; items inside a request's window are finished on the way (zeros)
    auto next_item = [&](int32_t item) -> Item {
      Item it;
      it.kind = 0;
      for (; item < n_items; item += stride) {
        it = decode_item(item, blk_prefix, n_req, n_kv_heads, G, window, cu_seqlens);
        if (it.kind == 2) break;
        if (wg == 0u && it.j0 + key < it.len) c_out[(int64_t)it.g * n_tokens + it.base + it.j0 + key] = 0.f;
        it.kind = 0;
      }
      if (it.kind == 2) it.w_inv = (uint32_t)(0x100000000ull / (uint32_t)it.w);
      return it;
    };
    uint32_t u0 = 0, nc = 0, n_own = 0;  // blocks before this item, items with products so far, this group's blocks so far
    bool ready = false;                 // my_lse[n_own & 1] already holds the log-sum-exp of the group's next block
    float lv[4];
    Item cur = next_item(item0);
    while (ok && cur.kind == 2) {
      const Item nxt = next_item(cur.number + stride);
      const uint32_t u1 = u0 + (uint32_t)cur.n_blocks;
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      for (int32_t t = (int32_t)((wg - u0) & 1u); t < cur.n_blocks; t += 2) {
        const uint32_t u = u0 + (uint32_t)t, lb = n_own & 1u;
        if (!ready) {
          fetch_lse(cur, t, lv);
#pragma unroll
          for (int c = 0; c < 4; ++c) my_lse[lb][32 * c + lane] = lv[c];
          __syncwarp();
        }
        // the group's next block, in this item or the next one: its log-sum-exp is in flight while this block is summed
        ready = true;
        if (t + 2 < cur.n_blocks) fetch_lse(cur, t + 2, lv);
        else if (nxt.kind == 2 && (int32_t)((wg - u1) & 1u) < nxt.n_blocks) fetch_lse(nxt, (int32_t)((wg - u1) & 1u), lv);
        else ready = false;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.d_full[wg]), (u >> 1) & 1u, abort_flag, wait_ns) ? 1 : 0) != 0;
        if (!ok) break;
        tc_fence_after();
        const float4* l4 = reinterpret_cast<const float4*>(my_lse[lb]);
        // the next 32 columns are on their way from TMEM while the current ones go through the exponentials
        uint32_t rr[2][32];
        tmem_ld32(t_lane + wg * kRows, rr[0]);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          tc_wait_ld();
          if (c + 1 < 4) tmem_ld32(t_lane + wg * kRows + 32 * (c + 1), rr[(c + 1) & 1]);
#pragma unroll
          for (int x = 0; x < 32; x += 4) {
            const float4 l = l4[8 * c + (x >> 2)];
            acc[0] += ex2(fmaf(__uint_as_float(rr[c & 1][x]), scale_log2, -l.x));
            acc[1] += ex2(fmaf(__uint_as_float(rr[c & 1][x + 1]), scale_log2, -l.y));
            if ((x >> 2) < kScorePoly) {
              // this pair's exponentials on the FMA pipe: the kernel is paced by the MUFU unit (one ex2 per logit)
              const float2 a = __ffma2_rn(make_float2(__uint_as_float(rr[c & 1][x + 2]), __uint_as_float(rr[c & 1][x + 3])),
                                          make_float2(scale_log2, scale_log2), make_float2(-l.z, -l.w));
              const float2 pp = exp2_poly2(a);
              acc[2] += pp.x;
              acc[3] += pp.y;
            } else {
              acc[2] += ex2(fmaf(__uint_as_float(rr[c & 1][x + 2]), scale_log2, -l.z));
              acc[3] += ex2(fmaf(__uint_as_float(rr[c & 1][x + 3]), scale_log2, -l.w));
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars.d_empty[wg]));
        if (ready) {
#pragma unroll
          for (int c = 0; c < 4; ++c) my_lse[lb ^ 1u][32 * c + lane] = lv[c];  // last read two of this warp's blocks ago
          __syncwarp();
        }
        ++n_own;
      }
      if (!ok) break;
      // the item's column sums: the second group hands its share over, the first adds and writes
      const float col_sum = (acc[0] + acc[1]) + (acc[2] + acc[3]);
      if (wg == 1u) {
        if (nc > 0u) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.comb_empty), (nc - 1u) & 1u, abort_flag, wait_ns) ? 1 : 0) != 0;
        if (!ok) break;
        comb_s[key] = col_sum;
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars.comb_full));
      } else {
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.comb_full), nc & 1u, abort_flag, wait_ns) ? 1 : 0) != 0;
        if (!ok) break;
        const float total = col_sum + comb_s[key];
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars.comb_empty));
        const int32_t j = cur.j0 + key;
        if (j < cur.len) c_out[(int64_t)cur.g * n_tokens + cur.base + j] = j < cur.nr ? total / (float)G : 0.f;
      }
      u0 = u1;
      ++nc;
      cur = nxt;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
  if (tid == 0 && abort_s && start_ok) atomicExch(status, (int32_t)PUREKV_ERR_TIMEOUT);
}


}  // namespace sc
}  // namespace purekv

using namespace purekv;

extern "C" purekv_status purekv_lowlayer_score_lse(const void* q, const void* k, const float* lse, float* c_out,
                                                   const purekv_batch* batch, int32_t window, int32_t n_q_heads,
                                                   int32_t n_kv_heads, int32_t head_dim, purekv_dtype dtype,
                                                   float softmax_scale, int32_t* status, void* stream) {
  using namespace sc;
  purekv_status st = check_batch(batch, true);
  if (st != PUREKV_OK) return st;
  if (batch->total_tokens == 0 || batch->n_req == 0) return PUREKV_OK;  // empty batch: nothing to do
  PK_REQUIRE(q && k && lse && c_out, PUREKV_ERR_INVALID_ARG, "purekv_lowlayer_score_lse: null pointer");
  PK_REQUIRE(n_q_heads >= 1 && n_kv_heads >= 1 && n_q_heads % n_kv_heads == 0, PUREKV_ERR_INVALID_ARG,
             "n_q_heads %d must be a positive multiple of n_kv_heads %d", n_q_heads, n_kv_heads);
  PK_REQUIRE(window >= 1, PUREKV_ERR_INVALID_ARG, "window must be >= 1");
  PK_REQUIRE(dtype == PUREKV_BF16 && head_dim == kD && window % 8 == 0, PUREKV_ERR_UNSUPPORTED,
             "purekv_lowlayer_score_lse needs bf16, head_dim 128 and a window that is a multiple of 8 "
             "(use purekv_lowlayer_score otherwise)");
  PK_REQUIRE(n_kv_heads <= 65535 && batch->n_req <= 65535, PUREKV_ERR_UNSUPPORTED, "too many heads or requests");
  PK_REQUIRE(((uintptr_t)q | (uintptr_t)k) % 16 == 0, PUREKV_ERR_INVALID_ARG, "Q/K must be 16-byte aligned");
  int32_t ml = 0;
  for (int r = 0; r < batch->n_req; ++r) {
    const int32_t len = batch->h_cu_seqlens[r + 1] - batch->h_cu_seqlens[r];
    ml = std::max(ml, len);
    // a request shorter than the window clips it; the clipped window must keep the boxes of rows inside one head
    PK_REQUIRE(len >= window || len % 8 == 0, PUREKV_ERR_UNSUPPORTED,
               "request %d: %d tokens, shorter than the window and not a multiple of 8", r, len);
  }
  // rows per box: the largest power of two up to 128 that divides the window of every request (clipped ones too)
  int32_t box_rows = kRows;
  while (window % box_rows) box_rows >>= 1;
  for (int r = 0; r < batch->n_req; ++r) {
    const int32_t len = batch->h_cu_seqlens[r + 1] - batch->h_cu_seqlens[r];
    if (len > 0 && len < window)
      while (len % box_rows) box_rows >>= 1;
  }
  const int64_t T = batch->total_tokens;
  CUtensorMap mk, mq8;
  if ((st = make_map(&mk, k, T, n_kv_heads, kKeys)) != PUREKV_OK) return st;
  if ((st = make_map(&mq8, q, T, n_q_heads, box_rows)) != PUREKV_OK) return st;
  if (!status) {
    const purekv_status st_w = default_status_word(&status);
    if (st_w != PUREKV_OK) return st_w;
  }
  const size_t smem = 1024 + (size_t)(1 + kStages) * kTile;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
  // Two forms.  One CTA per key block, handed out by the hardware over the grid (longest request's key blocks) x
  // heads x requests: a retiring CTA's successor starts while the SM's other CTA is in mid-item, which hides a CTA's
  // fixed costs well once an item has a few blocks of rows.  Two persistent CTAs per SM that take the items in turn
  // over the key blocks the requests really have: measured faster when an item is one or two blocks of rows (the
  // fixed costs were most of a CTA's time) and when the requests' lengths differ (the rectangular grid then launches
  // many CTAs that find nothing to do) unless the items are very long.
  const int64_t blocks_per_item = ((int64_t)(n_q_heads / n_kv_heads) * window + kRows - 1) / kRows;
  int64_t n_items = 0;  // the key blocks of every (request, KV head)
  for (int r = 0; r < batch->n_req; ++r)
    n_items += (int64_t)((batch->h_cu_seqlens[r + 1] - batch->h_cu_seqlens[r] + kKeys - 1) / kKeys) * n_kv_heads;
  if (n_items == 0) return PUREKV_OK;
  const int64_t n_rect = (int64_t)((ml + kKeys - 1) / kKeys) * n_kv_heads * batch->n_req;
  int dev = 0, n_sm = 0;
  PK_CUDA(cudaGetDevice(&dev));
  PK_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
  // (with no more than two items per persistent CTA there is nothing to overlap)
  const bool persistent = batch->n_req <= kMaxReq && n_items > 4 * (int64_t)n_sm &&
                          (blocks_per_item <= 2 || (n_items * 100 < n_rect * 85 && blocks_per_item < 20));
  if (!persistent) {
    static std::atomic<uint64_t> smem_allowed{0};
    const purekv_status st_smem = allow_max_dynamic_smem(score_tc_kernel, smem_allowed);
    if (st_smem != PUREKV_OK) return st_smem;
    dim3 grid((unsigned)((ml + kKeys - 1) / kKeys), (unsigned)n_kv_heads, (unsigned)batch->n_req);
    score_tc_kernel<<<grid, kThreads, smem, (cudaStream_t)stream>>>(mk, mq8, lse, c_out, batch->cu_seqlens, window,
                                                                     n_q_heads, n_kv_heads, scale * 1.4426950408889634f, T,
                                                                     status, wait_limit_ns(), box_rows);
  } else {
    static std::atomic<uint64_t> smem_allowed{0};
    const purekv_status st_smem = allow_max_dynamic_smem(score_tc_items_kernel, smem_allowed);
    if (st_smem != PUREKV_OK) return st_smem;
    PK_REQUIRE(n_items < (int64_t)1 << 30, PUREKV_ERR_UNSUPPORTED, "purekv_lowlayer_score_lse: %lld key blocks",
               (long long)n_items);
    dim3 grid((unsigned)std::min<int64_t>(n_items, 2 * (int64_t)n_sm));
    score_tc_items_kernel<<<grid, kThreads, smem, (cudaStream_t)stream>>>(
        mk, mq8, lse, c_out, batch->cu_seqlens, window, n_q_heads, n_kv_heads, scale * 1.4426950408889634f, T, status,
        wait_limit_ns(), box_rows, batch->n_req, (int32_t)n_items);
  }
  PK_CUDA(cudaGetLastError());
  return PUREKV_OK;
}
