// Internal interface between the prefill entry point and its two kernels.
#pragma once
#include "common.cuh"

namespace purekv {

struct PrefillArgs {
  const void *q, *k, *v;
  void* o;
  float* lse;
  const purekv_batch* batch;
  void* plan;
  const purekv_plan_info* info;
  int32_t n_q_heads, n_kv_heads, head_dim;
  purekv_dtype dtype;
  float scale;
  void* ws;
  size_t ws_bytes;
  int32_t* status;
  cudaStream_t stream;
};

purekv_status launch_prefill_simt(const PrefillArgs& a);  // CUDA cores: fp32, or bf16 with head_dim != 128
purekv_status launch_prefill_tc(const PrefillArgs& a);    // tcgen05 tensor cores: bf16, head_dim 128

}  // namespace purekv
