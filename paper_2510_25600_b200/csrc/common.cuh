// Shared host/device helpers of the PureKV CUDA library: error reporting,
// element-type conversion, and the plan buffer layout.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include "purekv.h"

namespace purekv {

void set_error(const char* fmt, ...);

#define PK_REQUIRE(cond, code, ...)         \
  do {                                      \
    if (!(cond)) {                          \
      ::purekv::set_error(__VA_ARGS__);     \
      return (code);                        \
    }                                       \
  } while (0)

#define PK_CUDA(expr)                                                                      \
  do {                                                                                     \
    cudaError_t e__ = (expr);                                                              \
    if (e__ != cudaSuccess) {                                                              \
      ::purekv::set_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__), __FILE__, \
                          __LINE__);                                                       \
      return PUREKV_ERR_CUDA;                                                              \
    }                                                                                      \
  } while (0)

purekv_status check_batch(const purekv_batch* b, bool need_device);
uint64_t wait_limit_ns();  // the process-wide limit of device-side waits (purekv_set_wait_limit_ns)

// The status word a call uses when the caller passes none: one word per device inside the library, read and
// cleared by purekv_poll_status(NULL, ...).  Its device address is looked up once per device.
purekv_status default_status_word(int32_t** out);

// Raises a kernel's dynamic shared-memory limit to what the device's opt-in maximum leaves, once per (kernel, device): `done`
// is a bit mask over device ordinals that the call site keeps in a function-local static.  Launches then pass
// whatever size they need; setting the attribute on every call would cost a driver call per launch.
template <typename Kernel>
purekv_status allow_max_dynamic_smem(Kernel kernel, std::atomic<uint64_t>& done) {
  int dev = -1;
  PK_CUDA(cudaGetDevice(&dev));
  PK_REQUIRE(dev >= 0 && dev < 64, PUREKV_ERR_UNSUPPORTED, "device ordinal %d is beyond 63", dev);
  if (done.load(std::memory_order_acquire) & (1ull << dev)) return PUREKV_OK;
  int max_optin = 0;
  PK_CUDA(cudaDeviceGetAttribute(&max_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
  cudaFuncAttributes fa;
  PK_CUDA(cudaFuncGetAttributes(&fa, kernel));  // the opt-in maximum covers the kernel's static shared memory too
  PK_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_optin - (int)fa.sharedSizeBytes));
  done.fetch_or(1ull << dev, std::memory_order_release);
  return PUREKV_OK;
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

// ---- plan buffer layout (device memory, written by purekv_plan_build) -------------------
// [PlanHeader][QTile x n_qtiles][order int32 x n_qtiles][entries int2 x n_entries][masks uint32 x n_mask_words]
// [Unit x n_units][merge counters int32 x n_counters][scheduling counters int32 x 2]
// all sections 16-byte aligned.  The last three sections exist only in plans for the tensor-core kernel, whose
// entries section also holds, behind the query tiles' own lists, the merged lists of the twin units (see Unit).
constexpr uint32_t kPlanMagic = 0x504B5636u;  // "PKV6"

// kTileNone appears only in the merged list of a twin unit: a key tile one of the two query tiles does not keep.
enum TileClass : int32_t { kTileFull = 0, kTileDiag = 1, kTileGeneral = 2, kTileNone = 3 };

struct PlanHeader {
  uint32_t magic;
  int32_t tile_q, tile_k;
  int32_t n_qtiles;
  int64_t total_tokens;
  int64_t n_entries;
  int64_t n_mask_words;
  int64_t off_qtiles, off_order, off_entries, off_masks;  // byte offsets from the plan base
  int32_t words_per_row;                                  // max(1, tile_k / 32)
  int32_t n_ctas, n_units, n_counters;
  int64_t off_units, off_counters;
  int32_t n_q_heads, n_kv_heads;
  int64_t part_slots;  // partial-result slots of the workspace (split chunks x query heads)
  uint32_t test_flags;  // 0 in every plan the planner writes; bit 0 (set by a test in a host copy of a plan): the
                        // producer withholds the first K copy, so that the bounded waits can be seen to expire
  uint32_t pad_flags;
};

struct QTile {
  int32_t q_start;      // absolute token index of the tile's first row
  int32_t q_rows;       // valid rows (<= tile_q)
  int32_t req_start;    // absolute token index of the request's first token
  int32_t req_len;
  int32_t entry_begin;  // into entries[]
  int32_t entry_count;
  int32_t pad[2];
};
// entry.x = (key tile index inside the request << 4) | (half mask << 2) | TileClass;  key tile kt covers
// request positions kt*tile_k .. kt*tile_k + tile_k - 1.  In tensor-core plans tile_k is 128 and, when the mask
// was built with a 64-key skip granularity, bit h of the half mask says whether keys 64h .. 64h+63 of the tile
// hold any kept pair (an absent half is neither loaded nor computed); otherwise the half mask is 3.
// entry.y = for a general tile, the index of its first mask word: row r of the query tile owns
// words [entry.y + r*words_per_row, +words_per_row), bit c of word w = key 32*w + c of the tile
// (causality already applied; rows past q_rows are zero); -1 otherwise.

// One unit of work of the tensor-core kernel: a query tile x a pair of query heads x a contiguous
// chunk of the tile's kept-key list.  The list is sorted by decreasing estimated cost; CTA c of n_ctas starts with
// unit c and draws further units (n_ctas, n_ctas + 1, ...) from the first scheduling counter as it finishes one;
// the second counts finished CTAs, and the last of them sets both back to zero.
// A list split into n_chunks > 1 chunks leaves one partial result per chunk and head in the
// workspace; the chunk that arrives last (merge counter) combines them.
//
// Twin units (q_rows1 > 0).  With an odd number G of query heads per KV head the last head of a group has no partner
// and its unit would leave half of the kernel idle.  Two consecutive query tiles of one request whose lists are
// cut into the same number of chunks share such a unit instead: both slots work on that head, slot 0 on the tile at
// q_start and slot 1 on the tile at q_start1, over the union of the two tiles' lists (of their chunks number
// `chunk`, when the lists are split; each tile keeps its own partial results and merge counters).  The union is stored as ent_count PAIRS of entries
// from ent_begin on: entries[ent_begin + 2n + s] is key tile n as slot s sees it, with its own class, half mask and
// bit mask, or class kTileNone with half mask 0 where that query tile keeps nothing of the key tile (the slot then
// multiplies by zeros).  The halves loaded and multiplied are the union of the two half masks.
struct __align__(16) Unit {
  int32_t q_start, q_rows, req_start;
  int32_t ent_begin, ent_count;  // into entries[]
  int32_t pair;                  // KV head g = pair / ppg, first query head g*G + 2*(pair % ppg), ppg = (G+1)/2
  int32_t chunk, n_chunks;
  int32_t part_base;             // workspace slot of (chunk 0, head 0) = part_base; slot(chunk, hq) = (part_base + chunk) * H + hq
  int32_t counter_base;          // merge counter of head hq = counters[counter_base + hq]
  int32_t q_start1, q_rows1;     // a twin unit's second query tile (q_rows1 == 0: an ordinary unit)
  int32_t part_base1, counter_base1;  // ... and that tile's workspace slots and merge counters when the lists are split
  int32_t pad[2];
};
static_assert(sizeof(Unit) == 64, "the plan's unit record is 16 words");

// Partial result of one (chunk, head): 128 x 128 fp32 unnormalised output laid out [col/4][row][col%4],
// then 128 reference maxima (log2 domain) and 128 row sums.
constexpr int64_t kPartFloats = 128 * 128 + 2 * 128;

}  // namespace purekv
