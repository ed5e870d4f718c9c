// purekv_decode_attention: one decoding step over the compacted cache of one layer (Sec. 3.1: later tokens attend
// to the compressed cache; the stage Table 3 times as decode latency).  Every request brings one new query per head;
// query head hq reads KV head hq / G of the request's kept rows.
//
// Split-KV, HBM bound: a CTA owns a chunk of one (request, KV head)'s kept keys and serves all G query heads of the
// group from one read of K and one of V.  Rows are 256 bytes (bf16 d = 128 or fp32 d = 64): a half-warp covers a
// row with one 16-byte load per lane, so a warp instruction fetches two rows.  Pass 1 forms the G logits of every
// key (q slices in registers; the 16 lanes' partial dot products are folded by a butterfly that halves the number of
// values per step) into shared memory; the chunk's maxima and exp2 weights are then taken once per element; pass 2
// streams V and accumulates G x d outputs in registers.  One chunk per (request, KV head): the CTA normalises and
// writes O itself; several: it leaves (unnormalised O, max, sum) per head and a second small kernel merges them.
#include <algorithm>

#include "common.cuh"

namespace purekv {

constexpr int kDecThreads = 128;
constexpr int kUnroll = 8;         // rows a half-warp has in flight
constexpr int kDecChunkMax = 512;  // keys per CTA: logits of 8 heads x 512 keys take 16 KB of shared memory

template <typename T>
struct Row16;  // the elements of one 16-byte chunk as fp32
template <>
struct Row16<float> {
  static constexpr int E = 4;
  static __device__ __forceinline__ void unpack(uint4 u, float (&f)[4]) {
    f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y); f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
  }
};
template <>
struct Row16<__nv_bfloat16> {
  static constexpr int E = 8;
  static __device__ __forceinline__ void unpack(uint4 u, float (&f)[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
};

__device__ __forceinline__ float dec_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Folds v[0..N) of the 16 lanes of a half-warp: each step a lane hands half of its values to the partner across
// `mask` and adds the partner's other half, so the values halve while the lanes summed double.  Afterwards v[0] of
// lane ch is the full 16-lane sum for head ch >> (4 - log2 N).
template <int N>
__device__ __forceinline__ void fold16(float (&v)[N], int ch) {
  int mask = 8;
  int n = N;
#pragma unroll
  for (int step = 0; step < 4; ++step) {
    if (n > 1) {
      const int half = n >> 1;
      const bool up = (ch & mask) != 0;
#pragma unroll
      for (int i = 0; i < N / 2; ++i) {
        if (i < half) {
          const float send = up ? v[i] : v[i + half];
          const float keep = up ? v[i + half] : v[i];
          v[i] = keep + __shfl_xor_sync(0xffffffffu, send, mask);
        }
      }
      n = half;
    } else {
      v[0] += __shfl_xor_sync(0xffffffffu, v[0], mask);
    }
    mask >>= 1;
  }
}

// grid (n_splits, H_kv, n_req), 128 threads.  part: [n_req][H][n_splits][D + 2] floats when n_splits > 1.
template <typename T, int GP>
__global__ void __launch_bounds__(kDecThreads) decode_partial_kernel(
    const uint4* __restrict__ q, const uint4* __restrict__ kc, const uint4* __restrict__ vc,
    const int32_t* __restrict__ cu_kept, int32_t n_q_heads, int32_t n_kv_heads, int32_t chunk, float scale_log2,
    T* __restrict__ o, float* __restrict__ lse, float* __restrict__ part, int32_t n_splits) {
  constexpr int E = Row16<T>::E, D = 16 * E;
  constexpr int kShift = GP == 8 ? 1 : GP == 4 ? 2 : GP == 2 ? 3 : 4;  // head of lane ch after fold16 = ch >> kShift
  __shared__ float s_sc[GP][kDecChunkMax];
  __shared__ float s_red[kDecThreads / 32][GP][D];
  __shared__ float s_m[GP], s_l[GP];

  const int32_t sp = blockIdx.x, g = blockIdx.y, r = blockIdx.z;
  const int32_t G = n_q_heads / n_kv_heads;
  const int32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, hw = lane >> 4, ch = lane & 15;
  const int64_t j0 = (int64_t)cu_kept[r] + (int64_t)sp * chunk;
  const int32_t n = (int32_t)max((int64_t)0, min((int64_t)cu_kept[r + 1], j0 + chunk) - j0);

  // this lane's slice of the group's queries, already in log2 units
  float qf[GP][E];
#pragma unroll
  for (int h = 0; h < GP; ++h) {
    float t[E];
#pragma unroll
    for (int e = 0; e < E; ++e) t[e] = 0.f;
    if (h < G) Row16<T>::unpack(__ldg(q + ((int64_t)r * n_q_heads + g * G + h) * 16 + ch), t);
#pragma unroll
    for (int e = 0; e < E; ++e) qf[h][e] = t[e] * scale_log2;
  }

  // pass 1: logits.  kUnroll rows per half-warp are requested before the first is used (bytes in flight); the bound
  // is rounded up to a pair of rows so that both halves of a warp make the same trips (the fold shuffles).
  constexpr int kStride = (kDecThreads / 32) * 2;
  const int32_t n_up = (n + 1) & ~1;
  for (int32_t p = warp * 2 + hw; p < n_up; p += kStride * kUnroll) {
    uint4 raw[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
      raw[u] = __ldg(kc + ((j0 + min(p + u * kStride, n - 1)) * n_kv_heads + g) * 16 + ch);
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int32_t pu = p + u * kStride;
      if (pu < n_up) {  // the same for every lane of the warp
        float kf[E];
        Row16<T>::unpack(raw[u], kf);
        float dot[GP];
#pragma unroll
        for (int h = 0; h < GP; ++h) {
          float a = 0.f;
#pragma unroll
          for (int e = 0; e < E; ++e) a = fmaf(qf[h][e], kf[e], a);
          dot[h] = a;
        }
        fold16<GP>(dot, ch);
        if ((ch & ((1 << kShift) - 1)) == 0 && pu < n) s_sc[ch >> kShift][pu] = dot[0];
      }
    }
  }
  __syncthreads();

  // per head: the chunk's maximum, then the weights 2^(s - max) in place and their sum (16 threads per head)
  {
    const int32_t h_t = tid >> 4, i0 = tid & 15;
    const int32_t h = min(h_t, GP - 1);  // surplus threads repeat the last head (whole warps stay in the shuffles)
    {
      float m = -INFINITY;
      for (int32_t i = i0; i < n; i += 16) m = fmaxf(m, s_sc[h][i]);
#pragma unroll
      for (int mask = 8; mask >= 1; mask >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, mask));
      float l = 0.f;
      for (int32_t i = i0; i < n; i += 16) {
        const float pw = dec_ex2(s_sc[h][i] - m);
        if (h_t < GP) s_sc[h][i] = pw;
        l += pw;
      }
#pragma unroll
      for (int mask = 8; mask >= 1; mask >>= 1) l += __shfl_xor_sync(0xffffffffu, l, mask);
      if (i0 == 0 && h_t < GP) {
        s_m[h] = m;
        s_l[h] = l;
      }
    }
  }
  __syncthreads();

  // pass 2: O += P V
  float acc[GP][E];
#pragma unroll
  for (int h = 0; h < GP; ++h)
#pragma unroll
    for (int e = 0; e < E; ++e) acc[h][e] = 0.f;
  for (int32_t p = warp * 2 + hw; p < n; p += kStride * kUnroll) {
    uint4 raw[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
      raw[u] = __ldg(vc + ((j0 + min(p + u * kStride, n - 1)) * n_kv_heads + g) * 16 + ch);
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int32_t pu = p + u * kStride;
      if (pu < n) {
        float vf[E];
        Row16<T>::unpack(raw[u], vf);
#pragma unroll
        for (int h = 0; h < GP; ++h) {
          const float pw = s_sc[h][pu];
#pragma unroll
          for (int e = 0; e < E; ++e) acc[h][e] = fmaf(pw, vf[e], acc[h][e]);
        }
      }
    }
  }
  // the two half-warps, then the four warps
#pragma unroll
  for (int h = 0; h < GP; ++h)
#pragma unroll
    for (int e = 0; e < E; ++e) acc[h][e] += __shfl_xor_sync(0xffffffffu, acc[h][e], 16);
  if (hw == 0) {
#pragma unroll
    for (int h = 0; h < GP; ++h)
#pragma unroll
      for (int e = 0; e < E; ++e) s_red[warp][h][ch * E + e] = acc[h][e];
  }
  __syncthreads();
  for (int32_t x = tid; x < G * D; x += kDecThreads) {
    const int32_t h = x / D, c = x % D;
    const float a = (s_red[0][h][c] + s_red[1][h][c]) + (s_red[2][h][c] + s_red[3][h][c]);
    const int32_t hq = g * G + h;
    if (n_splits == 1) {
      const float l = s_l[h];
      o[((int64_t)r * n_q_heads + hq) * D + c] = (T)(l > 0.f ? a / l : 0.f);
      if (c == 0 && lse) lse[(int64_t)r * n_q_heads + hq] = l > 0.f ? (s_m[h] + log2f(l)) * 0.6931471805599453f : -INFINITY;
    } else {
      float* dst = part + (((int64_t)r * n_q_heads + hq) * n_splits + sp) * (D + 2);
      dst[c] = a;
      if (c == 0) {
        dst[D] = s_m[h];
        dst[D + 1] = s_l[h];
      }
    }
  }
}

// grid (H, n_req), D threads: thread c merges column c of the splits' partial results.
template <typename T>
__global__ void decode_merge_kernel(const float* __restrict__ part, int32_t n_q_heads, int32_t n_splits, int32_t D,
                                    T* __restrict__ o, float* __restrict__ lse) {
  const int32_t hq = blockIdx.x, r = blockIdx.y, c = threadIdx.x;
  const float* src = part + ((int64_t)r * n_q_heads + hq) * n_splits * (D + 2);
  float m_all = -INFINITY;
  for (int32_t s = 0; s < n_splits; ++s)
    if (src[s * (D + 2) + D + 1] > 0.f) m_all = fmaxf(m_all, src[s * (D + 2) + D]);
  float a = 0.f, l = 0.f;
  for (int32_t s = 0; s < n_splits; ++s) {
    const float ls = src[s * (D + 2) + D + 1];
    if (ls > 0.f) {
      const float wgt = dec_ex2(src[s * (D + 2) + D] - m_all);
      a = fmaf(wgt, src[s * (D + 2) + c], a);
      l = fmaf(wgt, ls, l);
    }
  }
  o[((int64_t)r * n_q_heads + hq) * D + c] = (T)(l > 0.f ? a / l : 0.f);
  if (c == 0 && lse) lse[(int64_t)r * n_q_heads + hq] = l > 0.f ? (m_all + log2f(l)) * 0.6931471805599453f : -INFINITY;
}

// keys per CTA and CTAs per (request, KV head): enough CTAs for two per SM when the batch alone does not give them
// (more and shorter chunks were measured slower: the merge kernel walks a head's chunks one after the other)
static void decode_split(int32_t n_req, int32_t max_kept, int32_t n_kv_heads, int32_t* chunk, int32_t* n_splits) {
  const int64_t base = std::max<int64_t>(1, (int64_t)n_req * n_kv_heads);
  const int64_t want = std::max<int64_t>(1, (2 * 148 + base - 1) / base);
  int64_t c = (std::max(1, max_kept) + want - 1) / want;
  c = std::min<int64_t>(kDecChunkMax, std::max<int64_t>(64, c));
  c = (c + 7) / 8 * 8;
  *chunk = (int32_t)c;
  *n_splits = (int32_t)((std::max(1, max_kept) + c - 1) / c);
}

template <typename T, int GP>
static void launch_decode(dim3 grid, cudaStream_t sm, const void* q, const void* kc, const void* vc, const int32_t* cu_kept,
                          int32_t H, int32_t Hkv, int32_t chunk, float scale_log2, void* o, float* lse, float* part,
                          int32_t n_splits) {
  decode_partial_kernel<T, GP><<<grid, kDecThreads, 0, sm>>>((const uint4*)q, (const uint4*)kc, (const uint4*)vc, cu_kept, H,
                                                            Hkv, chunk, scale_log2, (T*)o, lse, part, n_splits);
}

}  // namespace purekv

using namespace purekv;

extern "C" {

size_t purekv_decode_ws_bytes(int32_t n_req, int32_t max_kept, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim) {
  if (n_req <= 0 || max_kept <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || head_dim <= 0) return 0;
  int32_t chunk, n_splits;
  decode_split(n_req, max_kept, n_kv_heads, &chunk, &n_splits);
  if (n_splits == 1) return 0;
  return (size_t)n_req * n_q_heads * n_splits * (head_dim + 2) * sizeof(float) + 256;
}

purekv_status purekv_decode_attention(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                                      const int32_t* cu_kept, const int32_t* h_cu_kept, int32_t n_req, int32_t n_q_heads,
                                      int32_t n_kv_heads, int32_t head_dim, purekv_dtype dtype, float softmax_scale,
                                      void* ws, size_t ws_bytes, void* stream) {
  PK_REQUIRE(n_req >= 0 && h_cu_kept, PUREKV_ERR_INVALID_ARG, "purekv_decode_attention: bad batch");
  PK_REQUIRE(n_q_heads > 0 && n_kv_heads > 0 && n_q_heads % n_kv_heads == 0, PUREKV_ERR_INVALID_ARG,
             "purekv_decode_attention: n_q_heads must be a positive multiple of n_kv_heads");
  PK_REQUIRE(dtype == PUREKV_BF16 || dtype == PUREKV_FP32, PUREKV_ERR_INVALID_ARG, "purekv_decode_attention: bad dtype");
  const int32_t G = n_q_heads / n_kv_heads;
  PK_REQUIRE((dtype == PUREKV_BF16 && head_dim == 128) || (dtype == PUREKV_FP32 && head_dim == 64), PUREKV_ERR_UNSUPPORTED,
             "purekv_decode_attention: rows must be 256 bytes (bf16 with head_dim 128, or fp32 with head_dim 64)");
  PK_REQUIRE(G <= 8, PUREKV_ERR_UNSUPPORTED, "purekv_decode_attention: at most 8 query heads per KV head");
  if (n_req == 0) return PUREKV_OK;
  int32_t max_kept = 0;
  PK_REQUIRE(h_cu_kept[0] == 0, PUREKV_ERR_INVALID_ARG, "purekv_decode_attention: cu_kept must start at 0");
  for (int32_t r = 0; r < n_req; ++r) {
    PK_REQUIRE(h_cu_kept[r + 1] >= h_cu_kept[r], PUREKV_ERR_INVALID_ARG, "purekv_decode_attention: cu_kept must not decrease");
    max_kept = std::max(max_kept, h_cu_kept[r + 1] - h_cu_kept[r]);
  }
  PK_REQUIRE(q && o && cu_kept, PUREKV_ERR_INVALID_ARG, "purekv_decode_attention: null pointer");
  PK_REQUIRE(h_cu_kept[n_req] == 0 || (k_cache && v_cache), PUREKV_ERR_INVALID_ARG, "purekv_decode_attention: null cache");
  PK_REQUIRE(((uintptr_t)q | (uintptr_t)k_cache | (uintptr_t)v_cache | (uintptr_t)o) % 16 == 0, PUREKV_ERR_INVALID_ARG,
             "purekv_decode_attention: pointers must be 16-byte aligned");
  int32_t chunk, n_splits;
  decode_split(n_req, max_kept, n_kv_heads, &chunk, &n_splits);
  float* part = nullptr;
  if (n_splits > 1) {
    PK_REQUIRE(ws && ws_bytes >= purekv_decode_ws_bytes(n_req, max_kept, n_q_heads, n_kv_heads, head_dim), PUREKV_ERR_WORKSPACE,
               "purekv_decode_attention: workspace of %zu bytes is too small", ws_bytes);
    part = (float*)(((uintptr_t)ws + 255) & ~(uintptr_t)255);
  }
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.f / sqrtf((float)head_dim);
  const float scale_log2 = scale * 1.4426950408889634f;
  cudaStream_t sm = (cudaStream_t)stream;
  dim3 grid((unsigned)n_splits, (unsigned)n_kv_heads, (unsigned)n_req);
  const int GP = G <= 1 ? 1 : G <= 2 ? 2 : G <= 4 ? 4 : 8;
#define PK_DECODE(T)                                                                                                     \
  switch (GP) {                                                                                                          \
    case 1: launch_decode<T, 1>(grid, sm, q, k_cache, v_cache, cu_kept, n_q_heads, n_kv_heads, chunk, scale_log2, o, lse, part, n_splits); break; \
    case 2: launch_decode<T, 2>(grid, sm, q, k_cache, v_cache, cu_kept, n_q_heads, n_kv_heads, chunk, scale_log2, o, lse, part, n_splits); break; \
    case 4: launch_decode<T, 4>(grid, sm, q, k_cache, v_cache, cu_kept, n_q_heads, n_kv_heads, chunk, scale_log2, o, lse, part, n_splits); break; \
    default: launch_decode<T, 8>(grid, sm, q, k_cache, v_cache, cu_kept, n_q_heads, n_kv_heads, chunk, scale_log2, o, lse, part, n_splits); break; \
  }
  if (dtype == PUREKV_BF16) {
    PK_DECODE(__nv_bfloat16)
  } else {
    PK_DECODE(float)
  }
#undef PK_DECODE
  PK_CUDA(cudaGetLastError());
  if (n_splits > 1) {
    dim3 g2((unsigned)n_q_heads, (unsigned)n_req);
    if (dtype == PUREKV_BF16)
      decode_merge_kernel<__nv_bfloat16><<<g2, head_dim, 0, sm>>>(part, n_q_heads, n_splits, head_dim, (__nv_bfloat16*)o, lse);
    else
      decode_merge_kernel<float><<<g2, head_dim, 0, sm>>>(part, n_q_heads, n_splits, head_dim, (float*)o, lse);
    PK_CUDA(cudaGetLastError());
  }
  return PUREKV_OK;
}

}  // extern "C"
