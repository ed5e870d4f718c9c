// Shared host/device helpers of the PureKV CUDA library: error reporting,
// element-type conversion, and the plan buffer layout.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

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

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

// ---- plan buffer layout (device memory, written by purekv_plan_build) -------------------
// [PlanHeader][QTile x n_qtiles][order int32 x n_qtiles][entries int2 x n_entries][masks uint32 x n_mask_words]
// all sections 16-byte aligned.
constexpr uint32_t kPlanMagic = 0x504B5632u;  // "PKV2"

enum TileClass : int32_t { kTileFull = 0, kTileDiag = 1, kTileGeneral = 2 };

struct PlanHeader {
  uint32_t magic;
  int32_t tile_q, tile_k;
  int32_t n_qtiles;
  int64_t total_tokens;
  int64_t n_entries;
  int64_t n_mask_words;
  int64_t off_qtiles, off_order, off_entries, off_masks;  // byte offsets from the plan base
  int32_t words_per_row;                                  // max(1, tile_k / 32)
  int32_t pad[3];
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
// entry.x = (key tile index inside the request << 2) | TileClass;  key tile kt covers request
// positions kt*tile_k .. kt*tile_k + tile_k - 1.
// entry.y = for a general tile, the index of its first mask word: row r of the query tile owns
// words [entry.y + r*words_per_row, +words_per_row), bit c of word w = key 32*w + c of the tile
// (causality already applied; rows past q_rows are zero); -1 otherwise.

}  // namespace purekv
