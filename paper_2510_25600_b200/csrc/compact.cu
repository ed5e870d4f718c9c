// purekv_compact_kv: gather of the surviving K/V rows into the compact cache (Sec. 3.1).
// One thread moves one 16-byte chunk of a K row and the matching chunk of the V row;
// consecutive threads write consecutive chunks of the output, so stores are fully coalesced
// and loads touch whole 32-byte sectors (a row is d * element size, a multiple of 16 bytes).
#include <algorithm>

#include "common.cuh"

namespace purekv {

__global__ void __launch_bounds__(256) compact_kernel(
    const uint4* __restrict__ k, const uint4* __restrict__ v, int64_t layer_stride_c /* chunks */,
    const int32_t* __restrict__ idx, const int32_t* __restrict__ cu_seqlens, const int32_t* __restrict__ cu_kept,
    int32_t n_req, int32_t k_tot, int32_t n_kv_heads, int32_t chunks_per_row, uint4* __restrict__ k_out,
    uint4* __restrict__ v_out, int64_t out_layer_stride_c, int64_t total_chunks_per_layer, int32_t n_layers) {
  // one-dimensional grid of at most one full wave; the threads stride over the chunks of all layers
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t total = total_chunks_per_layer * n_layers;
  for (int64_t xf = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; xf < total; xf += stride) {
    const int32_t layer = (int32_t)(xf / total_chunks_per_layer);
    const int64_t x = xf - layer * total_chunks_per_layer;
    const int32_t* idx_l = idx + (int64_t)layer * n_kv_heads * k_tot;
    const uint4* k_l = k + layer * layer_stride_c;
    const uint4* v_l = v + layer * layer_stride_c;
    uint4* ko = k_out + layer * out_layer_stride_c;
    uint4* vo = v_out + layer * out_layer_stride_c;
    const int32_t chunk = (int32_t)(x % chunks_per_row);
    const int64_t row = x / chunks_per_row;  // = t * n_kv_heads + g
    const int32_t g = (int32_t)(row % n_kv_heads);
    const int32_t t = (int32_t)(row / n_kv_heads);
    int32_t lo = 0, hi = n_req;  // request r with cu_kept[r] <= t < cu_kept[r+1]
    while (hi - lo > 1) {
      const int32_t mid = (lo + hi) >> 1;
      if (__ldg(cu_kept + mid) <= t) lo = mid; else hi = mid;
    }
    const int64_t src_tok = (int64_t)__ldg(cu_seqlens + lo) + __ldg(idx_l + (int64_t)g * k_tot + t);
    const int64_t src = (src_tok * n_kv_heads + g) * chunks_per_row + chunk;
    const uint4 kk = __ldg(k_l + src);
    const uint4 vv = __ldg(v_l + src);
    ko[x] = kk;
    vo[x] = vv;
  }
}

}  // namespace purekv

using namespace purekv;

extern "C" purekv_status purekv_compact_kv(const void* k, const void* v, int64_t layer_stride, int32_t n_layers,
                                           const int32_t* idx, const purekv_batch* batch, const int32_t* cu_kept,
                                           const int32_t* h_cu_kept, int32_t n_kv_heads, int32_t head_dim,
                                           purekv_dtype dtype, void* k_out, void* v_out, int64_t out_layer_stride,
                                           void* stream) {
  purekv_status st = check_batch(batch, true);
  if (st != PUREKV_OK) return st;
  if (batch->total_tokens == 0 || batch->n_req == 0) return PUREKV_OK;  // empty batch: nothing to do
  PK_REQUIRE(k && v && idx && cu_kept && h_cu_kept && k_out && v_out, PUREKV_ERR_INVALID_ARG,
             "purekv_compact_kv: null pointer");
  PK_REQUIRE(n_layers >= 0 && n_kv_heads >= 1 && head_dim >= 1, PUREKV_ERR_INVALID_ARG,
             "purekv_compact_kv: bad sizes");
  PK_REQUIRE(dtype == PUREKV_BF16 || dtype == PUREKV_FP32, PUREKV_ERR_INVALID_ARG, "unknown dtype");
  const int64_t esz = dtype == PUREKV_BF16 ? 2 : 4;
  const int64_t row_bytes = head_dim * esz;
  PK_REQUIRE(row_bytes % 16 == 0, PUREKV_ERR_UNSUPPORTED, "row of %lld bytes is not a multiple of 16",
             (long long)row_bytes);
  PK_REQUIRE((layer_stride * esz) % 16 == 0 && (out_layer_stride * esz) % 16 == 0, PUREKV_ERR_INVALID_ARG,
             "layer strides must be multiples of 16 bytes");
  PK_REQUIRE(((uintptr_t)k | (uintptr_t)v | (uintptr_t)k_out | (uintptr_t)v_out) % 16 == 0,
             PUREKV_ERR_INVALID_ARG, "K/V pointers must be 16-byte aligned");
  PK_REQUIRE(h_cu_kept[0] == 0, PUREKV_ERR_INVALID_ARG, "cu_kept[0] must be 0");
  for (int r = 0; r < batch->n_req; ++r) {
    const int32_t kr = h_cu_kept[r + 1] - h_cu_kept[r];
    PK_REQUIRE(kr >= 0 && kr <= batch->h_cu_seqlens[r + 1] - batch->h_cu_seqlens[r], PUREKV_ERR_INVALID_ARG,
               "request %d keeps %d rows of %d", r, kr, batch->h_cu_seqlens[r + 1] - batch->h_cu_seqlens[r]);
  }
  const int32_t k_tot = h_cu_kept[batch->n_req];
  PK_REQUIRE(layer_stride >= batch->total_tokens * n_kv_heads * head_dim || n_layers <= 1,
             PUREKV_ERR_INVALID_ARG, "layer_stride smaller than one layer");
  PK_REQUIRE(out_layer_stride >= (int64_t)k_tot * n_kv_heads * head_dim || n_layers <= 1,
             PUREKV_ERR_INVALID_ARG, "out_layer_stride smaller than one compacted layer");
  if (n_layers == 0 || k_tot == 0) return PUREKV_OK;
  const int32_t cpr = (int32_t)(row_bytes / 16);
  const int64_t per_layer = (int64_t)k_tot * n_kv_heads * cpr;
  const int64_t blocks = (per_layer * n_layers + 255) / 256;
  // one wave: 148 SMs x 8 resident CTAs of 256 threads; fewer blocks when the job is small
  dim3 grid((unsigned)std::min<int64_t>(blocks, 148 * 8));
  compact_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(
      (const uint4*)k, (const uint4*)v, layer_stride * esz / 16, idx, batch->cu_seqlens, cu_kept, batch->n_req, k_tot,
      n_kv_heads, cpr, (uint4*)k_out, (uint4*)v_out, out_layer_stride * esz / 16, per_layer, n_layers);
  PK_CUDA(cudaGetLastError());
  return PUREKV_OK;
}
