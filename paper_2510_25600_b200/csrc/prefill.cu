// purekv_st_sparse_prefill: argument checks and dispatch to the tensor-core or CUDA-core kernel.
#include "prefill.cuh"

using namespace purekv;

extern "C" purekv_status purekv_st_sparse_prefill(const void* q, const void* k, const void* v, void* o, float* lse,
                                                  const purekv_batch* batch, void* plan,
                                                  const purekv_plan_info* info, int32_t n_q_heads, int32_t n_kv_heads,
                                                  int32_t head_dim, purekv_dtype dtype, float softmax_scale, void* ws,
                                                  size_t ws_bytes, int32_t* status, void* stream) {
  purekv_status st = check_batch(batch, false);
  if (st != PUREKV_OK) return st;
  if (batch->total_tokens == 0 || batch->n_req == 0) return PUREKV_OK;  // empty batch: nothing to do
  PK_REQUIRE(q && k && v && o && plan && info, PUREKV_ERR_INVALID_ARG, "purekv_st_sparse_prefill: null pointer");
  PK_REQUIRE(n_q_heads >= 1 && n_kv_heads >= 1 && n_q_heads % n_kv_heads == 0 && n_q_heads <= 65535,
             PUREKV_ERR_INVALID_ARG, "n_q_heads %d must be a positive multiple of n_kv_heads %d", n_q_heads,
             n_kv_heads);
  PK_REQUIRE(dtype == PUREKV_BF16 || dtype == PUREKV_FP32, PUREKV_ERR_INVALID_ARG, "unknown dtype");
  PK_REQUIRE(info->dtype == (int32_t)dtype && info->head_dim == head_dim, PUREKV_ERR_INVALID_ARG,
             "plan was built for dtype %d head_dim %d, call has dtype %d head_dim %d", info->dtype, info->head_dim,
             (int)dtype, head_dim);
  PK_REQUIRE(info->n_q_heads == n_q_heads && info->n_kv_heads == n_kv_heads, PUREKV_ERR_INVALID_ARG,
             "plan was built for %d/%d heads, call has %d/%d", info->n_q_heads, info->n_kv_heads, n_q_heads,
             n_kv_heads);
  PK_REQUIRE(info->ws_bytes == 0 || (ws != nullptr && ws_bytes >= (size_t)info->ws_bytes && (uintptr_t)ws % 16 == 0),
             PUREKV_ERR_WORKSPACE, "prefill workspace: need %lld bytes (16-byte aligned), got %zu",
             (long long)info->ws_bytes, ws_bytes);
  PK_REQUIRE(((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)o | (uintptr_t)plan) % 16 == 0,
             PUREKV_ERR_INVALID_ARG, "Q/K/V/O/plan must be 16-byte aligned");
  if (info->n_qtiles == 0) return PUREKV_OK;
  PrefillArgs a{q, k, v, o, lse, batch, plan, info, n_q_heads, n_kv_heads, head_dim, dtype,
                softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim), ws, ws_bytes, status,
                (cudaStream_t)stream};
  if (dtype == PUREKV_BF16 && head_dim == 128 && info->tile_q == 128) return launch_prefill_tc(a);
  return launch_prefill_simt(a);
}
