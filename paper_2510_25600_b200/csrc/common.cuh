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
// [PlanHeader][QTile x n_qtiles][order int32 x n_qtiles][entries int32 x n_entries][meta int2 x T]
// all sections 16-byte aligned.
constexpr uint32_t kPlanMagic = 0x504B5631u;  // "PKV1"

enum TileClass : int32_t { kTileFull = 0, kTileDiag = 1, kTileGeneral = 2 };

struct PlanHeader {
  uint32_t magic;
  int32_t tile_q, tile_k;
  int32_t n_qtiles;
  int64_t total_tokens;
  int64_t n_entries;
  int64_t off_qtiles, off_order, off_entries, off_meta;  // byte offsets from the plan base
  // mask parameters the kernels evaluate for general tiles
  int32_t anchor_frames, spatial_radius, temporal_depth, temporal_stride, temporal_radius;
  int32_t dense_causal;
  int32_t pad[2];
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
// entry = (key tile index inside the request << 2) | TileClass;  key tile kt covers request
// positions kt*tile_k .. kt*tile_k + tile_k - 1.

// Per-token coordinates, int2:  x = kind | frame << 2 | (frame mod stride) << 17,  y = gy | gx << 16
// kind: 0 prefix text, 1 visual, 2 suffix text.
__host__ __device__ __forceinline__ int meta_kind(int mx) { return mx & 3; }
__host__ __device__ __forceinline__ int meta_frame(int mx) { return (mx >> 2) & 0x7FFF; }
__host__ __device__ __forceinline__ int meta_fmod(int mx) { return (mx >> 17) & 0x7FFF; }
__host__ __device__ __forceinline__ int meta_gy(int my) { return my & 0xFFFF; }
__host__ __device__ __forceinline__ int meta_gx(int my) { return (my >> 16) & 0xFFFF; }

struct MaskConsts {
  int32_t anchor_frames, spatial_radius, temporal_depth, temporal_stride, temporal_radius;
};

// Token-level mask of Sec. 3.2 for request-relative positions j <= i is checked by the caller.
// qm/km are the per-token coordinates of the query and the key.
__host__ __device__ __forceinline__ bool st_keep(const MaskConsts& mc, int2 qm, int2 km) {
  if (meta_kind(qm.x) != 1) return true;   // text query: dense
  if (meta_kind(km.x) == 0) return true;   // prefix key
  const int fq = meta_frame(qm.x), fk = meta_frame(km.x);
  if (fk < mc.anchor_frames) return true;  // first frame(s)
  const int dy = abs(meta_gy(qm.y) - meta_gy(km.y)), dx = abs(meta_gx(qm.y) - meta_gx(km.y));
  const int rho = dy > dx ? dy : dx;
  const int df = fq - fk;
  if (df == 0) return mc.spatial_radius < 0 || rho <= mc.spatial_radius;   // current frame
  const bool linked = meta_fmod(qm.x) == meta_fmod(km.x) &&
                      (mc.temporal_depth < 0 || df <= mc.temporal_depth * mc.temporal_stride);
  return linked && (mc.temporal_radius < 0 || rho <= mc.temporal_radius);  // previous frame(s)
}

}  // namespace purekv
