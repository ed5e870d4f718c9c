// purekv_lowlayer_score: window attention scores of the low layer (Eq. 1-2).
//
// For each request and KV head g the G*w query rows of the recent window (G query heads of
// the group x w positions) are stacked; row (hl, iw) is query head g*G+hl at position
// i = l-w+iw.  Pass 1 streams the keys once per 32-row block and keeps a running
// (max, sum of exponentials) per row -> log-sum-exp over all causal keys j <= i (Eq. 1's row
// normaliser).  Pass 2 gives each CTA one block of 64 non-recent keys: it recomputes the
// logits of every stacked row against those keys, forms exp(s - lse) and sums down the rows
// (Eq. 2), so the attention matrix never leaves the SM and no atomics are needed.
// Logits are fp32 FMA chains over exact products; exponentials use exp2f.
#include <algorithm>
#include <mutex>

#include "common.cuh"

namespace purekv {

// Scratch of purekv_lowlayer_score_noalloc: the window rows' log-sum-exp values and their per-key-block
// parts, i.e. what purekv_lowlayer_score keeps in its workspace.  It lives in the library's device image, so every GPU that
// loads the library holds this 1 MiB until the process exits.  Host code may not pass this name to
// a kernel (on the host it is only a stand-in for the symbol); the device address comes from
// cudaGetSymbolAddress, looked up once per device.
constexpr size_t kNoallocScoreFloats = PUREKV_NOALLOC_SCORE_MAX_ROWS;
static __device__ __align__(256) float g_noalloc_score_scratch[kNoallocScoreFloats + 64];  // + the 256 bytes of alignment slack the workspace rule asks for

constexpr int kRB = 32;        // stacked rows per block
constexpr int kKB = 64;        // keys per block
constexpr int kThreads = 256;  // thread (ty, tx): rows 2*ty, 2*ty+1; keys tx, tx+16, tx+32, tx+48

template <typename T>
__device__ __forceinline__ void load_row_f32(float* dst, const T* src, int d, int lane_in_group, int group_size) {
  for (int c = lane_in_group; c < d; c += group_size) dst[c] = to_f32(src[c]);
}

// s[a][b] = <q row 2*ty+a, key tx+16*b> over d, both tiles in shared memory with row stride ld.
__device__ __forceinline__ void tile_dots(const float* qs, const float* ks, int d, int ld, int ty, int tx,
                                          float s[2][4]) {
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) s[a][b] = 0.f;
  const float4* q0 = reinterpret_cast<const float4*>(qs + (2 * ty) * ld);
  const float4* q1 = reinterpret_cast<const float4*>(qs + (2 * ty + 1) * ld);
  for (int c = 0; c < d / 4; ++c) {
    const float4 a0 = q0[c], a1 = q1[c];
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const float4 kk = reinterpret_cast<const float4*>(ks + (tx + 16 * b) * ld)[c];
      s[0][b] = fmaf(a0.x, kk.x, s[0][b]);
      s[0][b] = fmaf(a0.y, kk.y, s[0][b]);
      s[0][b] = fmaf(a0.z, kk.z, s[0][b]);
      s[0][b] = fmaf(a0.w, kk.w, s[0][b]);
      s[1][b] = fmaf(a1.x, kk.x, s[1][b]);
      s[1][b] = fmaf(a1.y, kk.y, s[1][b]);
      s[1][b] = fmaf(a1.z, kk.z, s[1][b]);
      s[1][b] = fmaf(a1.w, kk.w, s[1][b]);
    }
  }
}

// Pass 1.  grid (row blocks, n_kv_heads, n_req).  lse2 [n_req][H][window] in log2 units of the
// scaled logits (s * scale * log2 e).
template <typename T>
__global__ void __launch_bounds__(kThreads) score_lse_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                             const int32_t* __restrict__ cu_seqlens, int32_t window,
                                                             int32_t n_q_heads, int32_t n_kv_heads, int32_t d,
                                                             float scale_log2, float* __restrict__ lse2) {
  extern __shared__ __align__(16) float smem[];
  const int ld = d + 4;
  float* qs = smem;             // [kRB][ld]
  float* ks = smem + kRB * ld;  // [kKB][ld]
  const int32_t r = blockIdx.z, g = blockIdx.y;
  const int32_t G = n_q_heads / n_kv_heads;
  const int32_t base = cu_seqlens[r], len = cu_seqlens[r + 1] - base;
  const int32_t w = min(window, len);
  const int32_t n_rows = G * w;
  const int32_t row0 = blockIdx.x * kRB;
  if (row0 >= n_rows) return;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  // stage the query rows (rows past n_rows are zero)
  for (int rr = tid >> 3; rr < kRB; rr += kThreads / 8) {
    const int32_t row = row0 + rr;
    float* dst = qs + rr * ld;
    if (row < n_rows) {
      const int32_t hq = g * G + row / w, i = len - w + row % w;
      load_row_f32(dst, q + ((int64_t)(base + i) * n_q_heads + hq) * d, d, tid & 7, 8);
    } else {
      for (int c = tid & 7; c < d; c += 8) dst[c] = 0.f;
    }
  }
  int32_t my_i[2];
#pragma unroll
  for (int a = 0; a < 2; ++a) {
    const int32_t row = row0 + 2 * ty + a;
    my_i[a] = row < n_rows ? len - w + row % w : -1;
  }
  // last key any row of this block needs
  const int32_t last_row = min(n_rows, row0 + kRB) - 1;
  int32_t i_max = 0;
  if (row0 / w == last_row / w) i_max = len - w + last_row % w; else i_max = len - 1;
  float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
  for (int32_t j0 = 0; j0 <= i_max; j0 += kKB) {
    __syncthreads();
    for (int rr = tid >> 3; rr < kKB; rr += kThreads / 8) {
      const int32_t j = j0 + rr;
      float* dst = ks + rr * ld;
      if (j < len) load_row_f32(dst, k + ((int64_t)(base + j) * n_kv_heads + g) * d, d, tid & 7, 8);
      else for (int c = tid & 7; c < d; c += 8) dst[c] = 0.f;
    }
    __syncthreads();
    float s[2][4];
    tile_dots(qs, ks, d, ld, ty, tx, s);
#pragma unroll
    for (int a = 0; a < 2; ++a) {
      float tmax = -INFINITY;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int32_t j = j0 + tx + 16 * b;
        s[a][b] = j <= my_i[a] ? s[a][b] * scale_log2 : -INFINITY;
        tmax = fmaxf(tmax, s[a][b]);
      }
      if (tmax > -INFINITY) {
        const float mn = fmaxf(m[a], tmax);
        float add = 0.f;
#pragma unroll
        for (int b = 0; b < 4; ++b) add += exp2f(s[a][b] - mn);
        l[a] = l[a] * exp2f(m[a] - mn) + add;
        m[a] = mn;
      }
    }
  }
  // combine the 16 threads (tx) that share a row: lanes differ in the low 4 bits
#pragma unroll
  for (int a = 0; a < 2; ++a) {
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) {
      const float mo = __shfl_xor_sync(0xffffffffu, m[a], off), lo = __shfl_xor_sync(0xffffffffu, l[a], off);
      const float mn = fmaxf(m[a], mo);
      if (mn > -INFINITY) {
        l[a] = l[a] * exp2f(m[a] - mn) + lo * exp2f(mo - mn);
        m[a] = mn;
      }
    }
    const int32_t row = row0 + 2 * ty + a;
    if (tx == 0 && row < n_rows)
      lse2[((int64_t)r * n_q_heads + g * G + row / w) * window + row % w] = m[a] + log2f(l[a]);
  }
}

// Pass 2.  grid (key blocks over the longest request, n_kv_heads, n_req).
template <typename T>
__global__ void __launch_bounds__(kThreads) score_colsum_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                                const int32_t* __restrict__ cu_seqlens,
                                                                int32_t window, int32_t obs, int32_t n_q_heads,
                                                                int32_t n_kv_heads, int32_t d, float scale_log2,
                                                                const float* __restrict__ lse2, int64_t n_tokens,
                                                                float* __restrict__ c_out) {
  extern __shared__ __align__(16) float smem[];
  __shared__ float red[kThreads / 16][kKB];
  const int ld = d + 4;
  float* qs = smem;
  float* ks = smem + kRB * ld;
  const int32_t r = blockIdx.z, g = blockIdx.y;
  const int32_t G = n_q_heads / n_kv_heads;
  const int32_t base = cu_seqlens[r], len = cu_seqlens[r + 1] - base;
  const int32_t w = min(window, len);
  const int32_t nr = len - w;  // non-recent keys
  const int32_t wo = min(obs, len);  // rows that are accumulated: the last wo of the request (Eq. 2: wo = w)
  const int32_t j0 = blockIdx.x * kKB;
  if (j0 >= len) return;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  float* cg = c_out + (int64_t)g * n_tokens + base;
  if (j0 >= nr) {  // block inside the window: defined as 0
    for (int c = tid; c < kKB; c += kThreads)
      if (j0 + c < len) cg[j0 + c] = 0.f;
    return;
  }
  for (int rr = tid >> 3; rr < kKB; rr += kThreads / 8) {
    const int32_t j = j0 + rr;
    float* dst = ks + rr * ld;
    if (j < len) load_row_f32(dst, k + ((int64_t)(base + j) * n_kv_heads + g) * d, d, tid & 7, 8);
    else for (int c = tid & 7; c < d; c += 8) dst[c] = 0.f;
  }
  const int32_t n_rows = G * wo;
  float col[4] = {0.f, 0.f, 0.f, 0.f};
  for (int32_t row0 = 0; row0 < n_rows; row0 += kRB) {
    __syncthreads();
    for (int rr = tid >> 3; rr < kRB; rr += kThreads / 8) {
      const int32_t row = row0 + rr;
      float* dst = qs + rr * ld;
      if (row < n_rows) {
        const int32_t hq = g * G + row / wo, i = len - wo + row % wo;
        load_row_f32(dst, q + ((int64_t)(base + i) * n_q_heads + hq) * d, d, tid & 7, 8);
      } else {
        for (int c = tid & 7; c < d; c += 8) dst[c] = 0.f;
      }
    }
    __syncthreads();
    float s[2][4];
    tile_dots(qs, ks, d, ld, ty, tx, s);
#pragma unroll
    for (int a = 0; a < 2; ++a) {
      const int32_t row = row0 + 2 * ty + a;
      if (row < n_rows) {
        const float lse = __ldg(lse2 + ((int64_t)r * n_q_heads + g * G + row / wo) * obs + row % wo);
        // with wo = w every non-recent key precedes every accumulated row; a longer observation reaches rows that
        // lie before some of the block's keys, and a row only counts for the keys it can see
        const int32_t i = len - wo + row % wo;
#pragma unroll
        for (int b = 0; b < 4; ++b)
          if (j0 + tx + 16 * b <= i) col[b] += exp2f(s[a][b] * scale_log2 - lse);
      }
    }
  }
#pragma unroll
  for (int b = 0; b < 4; ++b) red[ty][tx + 16 * b] = col[b];
  __syncthreads();
  if (tid < kKB) {
    float sum = 0.f;
#pragma unroll
    for (int t = 0; t < kThreads / 16; ++t) sum += red[t][tid];
    const int32_t j = j0 + tid;
    if (j < len) cg[j] = j < nr ? sum / (float)G : 0.f;
  }
}

static int32_t max_len(const purekv_batch* b) {
  int32_t m = 0;
  for (int r = 0; r < b->n_req; ++r) m = std::max(m, b->h_cu_seqlens[r + 1] - b->h_cu_seqlens[r]);
  return m;
}

// ---- bf16 path on tensor cores ------------------------------------------------------------------
// Both passes use the same tiling: a CTA owns one block of 128 keys of one (request, KV head) and walks the
// G*w stacked window rows in blocks of 128; its 8 warps form a 4 x 2 grid, warp (wr, wc) computing the 32 x 64
// logits of rows 32*wr .. +31 against keys 64*wc .. +63 with mma.sync m16n8k16 (bf16 x bf16 -> fp32: products
// exact, fp32 accumulation).  Pass 1 leaves, per 64-key block and row, the maximum and the sum of exponentials of
// the causal logits; a small kernel folds those into the row's log-sum-exp; pass 2 forms exp(s - lse) and sums down
// the rows.  Every key block is an independent CTA, so the grid is (key blocks) x (KV heads) x (requests) in both
// passes.
constexpr int kMmaKeys = 64;    // keys per warp column, and the granularity of the pass-1 (max, sum) pairs
constexpr int kCtaKeys = 128;   // keys per CTA
constexpr int kMmaRows = 128;
constexpr int kMmaThreads = 256;

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t addr, uint32_t (&r)[2]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16x8x16(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// Copies `rows` rows of d bf16 (global row r at src + row_of(r)) into shared memory with a row stride of d + 8
// elements (conflict-free for ldmatrix); rows for which row_of gives a negative offset are zero-filled.
template <typename RowOf>
__device__ __forceinline__ void stage_rows_bf16(__nv_bfloat16* dst, const __nv_bfloat16* src, int rows, int d, RowOf row_of) {
  const int cpr = d / 8;  // 16-byte chunks per row
  for (int x = threadIdx.x; x < rows * cpr; x += kMmaThreads) {
    const int r = x / cpr, c = x % cpr;
    const int64_t off = row_of(r);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (off >= 0) v = __ldg(reinterpret_cast<const uint4*>(src + off) + c);
    *reinterpret_cast<uint4*>(dst + r * (d + 8) + c * 8) = v;
  }
}

// The same copy with cp.async (16 bytes per request, zero fill for absent rows): returns at once, the data is
// there after cp_async_wait.  Used to load the next block of query rows while the current one is multiplied.
template <typename RowOf>
__device__ __forceinline__ void stage_rows_bf16_async(__nv_bfloat16* dst, const __nv_bfloat16* src, int rows, int d, RowOf row_of) {
  const int cpr = d / 8;
  for (int x = threadIdx.x; x < rows * cpr; x += kMmaThreads) {
    const int r = x / cpr, c = x % cpr;
    const int64_t off = row_of(r);
    const uint32_t sa = (uint32_t)__cvta_generic_to_shared(dst + r * (d + 8) + c * 8);
    const void* ga = off >= 0 ? (const void*)(reinterpret_cast<const uint4*>(src + off) + c) : (const void*)src;
    const uint32_t bytes = off >= 0 ? 16u : 0u;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(sa), "l"(ga), "r"(bytes) : "memory");
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// acc[mb][nb][0..3] = logits of rows (32*wr + 16*mb + lane/4, +8) x keys (64*wc + 8*nb + 2*(lane%4), +1) of the
// staged tiles: per 16-wide K step two A fragments and four ldmatrix.x4 of K feed sixteen MMAs.
__device__ __forceinline__ void logits_32x64(const __nv_bfloat16* qs, const __nv_bfloat16* ks, int d, float (&acc)[2][8][4]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wr = warp >> 1, wc = warp & 1, ld = d + 8;
#pragma unroll
  for (int mb = 0; mb < 2; ++mb)
#pragma unroll
    for (int nb = 0; nb < 8; ++nb)
#pragma unroll
      for (int x = 0; x < 4; ++x) acc[mb][nb][x] = 0.f;
  const uint32_t qa = (uint32_t)__cvta_generic_to_shared(qs + (32 * wr + (lane & 7) + 8 * ((lane >> 3) & 1)) * ld + 8 * (lane >> 4));
  // K: one x4 covers two 8-key blocks: matrices (keys +0, k 0-7), (keys +0, k 8-15), (keys +8, k 0-7), (keys +8, k 8-15)
  const uint32_t ka = (uint32_t)__cvta_generic_to_shared(ks + (64 * wc + (lane & 7) + 8 * (lane >> 4)) * ld + 8 * ((lane >> 3) & 1));
  for (int k0 = 0; k0 < d; k0 += 16) {
    uint32_t a0[4], a1[4];
    ldmatrix_x4(qa + k0 * 2, a0);
    ldmatrix_x4(qa + (16 * ld + k0) * 2, a1);
#pragma unroll
    for (int nb = 0; nb < 8; nb += 2) {
      uint32_t b4[4];
      ldmatrix_x4(ka + (nb * 8 * ld + k0) * 2, b4);
      const uint32_t b0[2] = {b4[0], b4[1]}, b1[2] = {b4[2], b4[3]};
      mma_bf16_16x8x16(acc[0][nb], a0, b0);
      mma_bf16_16x8x16(acc[1][nb], a1, b0);
      mma_bf16_16x8x16(acc[0][nb + 1], a0, b1);
      mma_bf16_16x8x16(acc[1][nb + 1], a1, b1);
    }
  }
}

// Pass 1.  partial[((r * Hkv + g) * n_kb + kb64) * rows_max + row] = (max, sum of exp2) of the causal logits of the
// stacked row against the 64-key block kb64, in log2 units of the scaled logits.
__global__ void __launch_bounds__(kMmaThreads) score_mma_partial_kernel(
    const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k, const int32_t* __restrict__ cu_seqlens,
    int32_t window, int32_t n_q_heads, int32_t n_kv_heads, int32_t d, float scale_log2, int32_t n_kb, int32_t rows_max,
    float2* __restrict__ partial) {
  extern __shared__ __align__(16) uint8_t smem_mma[];
  __nv_bfloat16* ks = reinterpret_cast<__nv_bfloat16*>(smem_mma);
  __nv_bfloat16* qs = ks + kCtaKeys * (d + 8);
  const int32_t r = blockIdx.z, g = blockIdx.y;
  const int32_t G = n_q_heads / n_kv_heads;
  const int32_t base = cu_seqlens[r], len = cu_seqlens[r + 1] - base;
  const int32_t w = min(window, len), n_rows = G * w, j0 = blockIdx.x * kCtaKeys;
  if (j0 >= len) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wr = warp >> 1, wc = warp & 1;
  stage_rows_bf16(ks, k, kCtaKeys, d, [&](int rr) -> int64_t {
    return j0 + rr < len ? ((int64_t)(base + j0 + rr) * n_kv_heads + g) * d : -1;
  });
  const int32_t kb64 = 2 * blockIdx.x + wc;  // this warp's 64-key block
  float2* out = partial + ((int64_t)(r * n_kv_heads + g) * n_kb + kb64) * rows_max;
  const bool block_live = j0 + 64 * wc < len;  // the second half of the last CTA may lie past the request
  auto q_row = [&](int32_t row) -> int64_t {
    return row < n_rows ? ((int64_t)(base + len - w + row % w) * n_q_heads + g * G + row / w) * d : -1;
  };
  __nv_bfloat16* qbuf[2] = {qs, qs + kMmaRows * (d + 8)};
  stage_rows_bf16_async(qbuf[0], q, kMmaRows, d, [&](int rr) { return q_row(rr); });
  for (int32_t row0 = 0, it = 0; row0 < n_rows; row0 += kMmaRows, ++it) {
    __syncthreads();  // everyone is done with the buffer the next copy overwrites (and, first time, K is staged)
    if (row0 + kMmaRows < n_rows) {
      stage_rows_bf16_async(qbuf[(it + 1) & 1], q, kMmaRows, d, [&](int rr) { return q_row(row0 + kMmaRows + rr); });
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const __nv_bfloat16* qcur = qbuf[it & 1];
    float acc[2][8][4];
    logits_32x64(qcur, ks, d, acc);
#pragma unroll
    for (int mb = 0; mb < 2; ++mb)
#pragma unroll
      for (int h = 0; h < 2; ++h) {  // the thread's four rows
        const int32_t row = row0 + 32 * wr + 16 * mb + (lane >> 2) + 8 * h;
        const int32_t i = row < n_rows ? len - w + row % w : -1;  // causal limit of the row (-1: no row)
        float m = -INFINITY;
#pragma unroll
        for (int nb = 0; nb < 8; ++nb)
#pragma unroll
          for (int x = 0; x < 2; ++x) {
            const int32_t j = j0 + 64 * wc + 8 * nb + 2 * (lane & 3) + x;
            const float sv = j <= i ? acc[mb][nb][2 * h + x] * scale_log2 : -INFINITY;
            acc[mb][nb][2 * h + x] = sv;
            m = fmaxf(m, sv);
          }
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
        float l = 0.f;
        if (m > -INFINITY) {
#pragma unroll
          for (int nb = 0; nb < 8; ++nb) l += exp2f(acc[mb][nb][2 * h] - m) + exp2f(acc[mb][nb][2 * h + 1] - m);
        }
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        if ((lane & 3) == 0 && row < n_rows && block_live) out[row] = make_float2(m, l);
      }
  }
}

// Folds the per-key-block (max, sum) pairs into each stacked row's log-sum-exp.  One thread per (request, query
// head, window position).
__global__ void __launch_bounds__(256) score_lse_merge_kernel(const float2* __restrict__ partial,
                                                              const int32_t* __restrict__ cu_seqlens, int32_t window,
                                                              int32_t n_q_heads, int32_t n_kv_heads, int32_t n_kb,
                                                              int32_t rows_max, int32_t n_req, float* __restrict__ lse2) {
  const int64_t x = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= (int64_t)n_req * n_q_heads * window) return;
  const int32_t iw = (int32_t)(x % window), hq = (int32_t)((x / window) % n_q_heads), r = (int32_t)(x / ((int64_t)window * n_q_heads));
  const int32_t G = n_q_heads / n_kv_heads, g = hq / G, hl = hq % G;
  const int32_t len = cu_seqlens[r + 1] - cu_seqlens[r];
  const int32_t w = min(window, len);
  if (iw >= w) return;
  const int32_t row = hl * w + iw, kbs = (len + kMmaKeys - 1) / kMmaKeys;
  const float2* p = partial + ((int64_t)(r * n_kv_heads + g) * n_kb) * rows_max + row;
  float m = -INFINITY;
  for (int32_t kb = 0; kb < kbs; ++kb) m = fmaxf(m, p[(int64_t)kb * rows_max].x);
  float l = 0.f;
  for (int32_t kb = 0; kb < kbs; ++kb) {
    const float2 v = p[(int64_t)kb * rows_max];
    if (v.y > 0.f) l += v.y * exp2f(v.x - m);
  }
  lse2[((int64_t)r * n_q_heads + hq) * window + iw] = m + log2f(l);
}

// Pass 2 (Eq. 2).  C[g, j] = (1/G) * sum over the stacked rows of exp2(s - lse) for the non-recent keys of the CTA's block.
__global__ void __launch_bounds__(kMmaThreads) score_mma_colsum_kernel(
    const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k, const int32_t* __restrict__ cu_seqlens,
    int32_t window, int32_t obs, int32_t n_q_heads, int32_t n_kv_heads, int32_t d, float scale_log2,
    const float* __restrict__ lse2, int64_t n_tokens, float* __restrict__ c_out) {
  extern __shared__ __align__(16) uint8_t smem_mma[];
  __shared__ float red[4][kCtaKeys];  // per row group of warps
  __nv_bfloat16* ks = reinterpret_cast<__nv_bfloat16*>(smem_mma);
  __nv_bfloat16* qs = ks + kCtaKeys * (d + 8);
  const int32_t r = blockIdx.z, g = blockIdx.y, j0 = blockIdx.x * kCtaKeys;
  const int32_t G = n_q_heads / n_kv_heads;
  const int32_t base = cu_seqlens[r], len = cu_seqlens[r + 1] - base;
  const int32_t w = min(window, len), nr = len - w;
  const int32_t wo = min(obs, len), n_rows = G * wo;  // accumulated rows: the last wo of the request (Eq. 2: wo = w)
  if (j0 >= len) return;
  float* cg = c_out + (int64_t)g * n_tokens + base;
  if (j0 >= nr) {  // block inside the window: defined as 0
    for (int c = threadIdx.x; c < kCtaKeys; c += kMmaThreads)
      if (j0 + c < len) cg[j0 + c] = 0.f;
    return;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wr = warp >> 1, wc = warp & 1;
  stage_rows_bf16(ks, k, kCtaKeys, d, [&](int rr) -> int64_t {
    return j0 + rr < len ? ((int64_t)(base + j0 + rr) * n_kv_heads + g) * d : -1;
  });
  float col[8][2];
#pragma unroll
  for (int nb = 0; nb < 8; ++nb) col[nb][0] = col[nb][1] = 0.f;
  auto q_row = [&](int32_t row) -> int64_t {
    return row < n_rows ? ((int64_t)(base + len - wo + row % wo) * n_q_heads + g * G + row / wo) * d : -1;
  };
  __nv_bfloat16* qbuf[2] = {qs, qs + kMmaRows * (d + 8)};
  stage_rows_bf16_async(qbuf[0], q, kMmaRows, d, [&](int rr) { return q_row(rr); });
  for (int32_t row0 = 0, it = 0; row0 < n_rows; row0 += kMmaRows, ++it) {
    __syncthreads();  // everyone is done with the buffer the next copy overwrites (and, first time, K is staged)
    if (row0 + kMmaRows < n_rows) {
      stage_rows_bf16_async(qbuf[(it + 1) & 1], q, kMmaRows, d, [&](int rr) { return q_row(row0 + kMmaRows + rr); });
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const __nv_bfloat16* qcur = qbuf[it & 1];
    float acc[2][8][4];
    logits_32x64(qcur, ks, d, acc);
#pragma unroll
    for (int mb = 0; mb < 2; ++mb)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int32_t row = row0 + 32 * wr + 16 * mb + (lane >> 2) + 8 * h;
        if (row < n_rows) {
          const float lse = __ldg(lse2 + ((int64_t)r * n_q_heads + g * G + row / wo) * obs + row % wo);
          if (wo == w) {
            // every non-recent key precedes every window row, so causality holds for all of them
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) {
              col[nb][0] += exp2f(fmaf(acc[mb][nb][2 * h], scale_log2, -lse));
              col[nb][1] += exp2f(fmaf(acc[mb][nb][2 * h + 1], scale_log2, -lse));
            }
          } else {
            // a longer observation reaches rows that lie before some keys: a row only counts for the keys it sees
            const int32_t i = len - wo + row % wo, jb = j0 + 64 * wc + 2 * (lane & 3);
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) {
              if (jb + 8 * nb <= i) col[nb][0] += exp2f(fmaf(acc[mb][nb][2 * h], scale_log2, -lse));
              if (jb + 8 * nb + 1 <= i) col[nb][1] += exp2f(fmaf(acc[mb][nb][2 * h + 1], scale_log2, -lse));
            }
          }
        }
      }
  }
  // sum over the 8 row groups of the warp (lanes with equal lane % 4 hold the same columns), then over the 4 row warps
#pragma unroll
  for (int nb = 0; nb < 8; ++nb)
#pragma unroll
    for (int x = 0; x < 2; ++x) {
      float v = col[nb][x];
      v += __shfl_xor_sync(0xffffffffu, v, 4);
      v += __shfl_xor_sync(0xffffffffu, v, 8);
      v += __shfl_xor_sync(0xffffffffu, v, 16);
      if (lane < 4) red[wr][64 * wc + 8 * nb + 2 * lane + x] = v;
    }
  __syncthreads();
  if (threadIdx.x < kCtaKeys) {
    const float sum = (red[0][threadIdx.x] + red[1][threadIdx.x]) + (red[2][threadIdx.x] + red[3][threadIdx.x]);
    const int32_t j = j0 + threadIdx.x;
    if (j < len) cg[j] = j < nr ? sum / (float)G : 0.f;
  }
}

// `obs` = accumulated rows per request and head (Eq. 2: the window itself); the first pass and the merge see only
// rows, so they take it in place of the window.
static purekv_status launch_score_mma(const void* q, const void* k, float* c_out, const purekv_batch* b, int32_t window,
                                      int32_t obs, int32_t H, int32_t Hkv, int32_t d, float scale, float* ws_f,
                                      cudaStream_t sm) {
  const int32_t ml = max_len(b);
  const int32_t n_kb = (ml + kMmaKeys - 1) / kMmaKeys, rows_max = (H / Hkv) * obs;
  float* lse2 = ws_f;                                                             // [n_req][H][obs]
  // the pairs start on a 256-byte boundary behind the log-sum-exp values
  float2* partial = reinterpret_cast<float2*>(ws_f + (((int64_t)b->n_req * H * obs + 63) & ~(int64_t)63));  // [n_req][Hkv][n_kb][rows_max]
  const size_t smem = (size_t)(kCtaKeys + 2 * kMmaRows) * (d + 8) * sizeof(__nv_bfloat16);  // K block + two Q blocks
  {
    static std::atomic<uint64_t> smem_allowed{0};
    const purekv_status st_smem = allow_max_dynamic_smem(score_mma_partial_kernel, smem_allowed);
    if (st_smem != PUREKV_OK) return st_smem;
  }
  {
    static std::atomic<uint64_t> smem_allowed{0};
    const purekv_status st_smem = allow_max_dynamic_smem(score_mma_colsum_kernel, smem_allowed);
    if (st_smem != PUREKV_OK) return st_smem;
  }
  const float scale_log2 = scale * 1.4426950408889634f;
  dim3 grid((unsigned)((ml + kCtaKeys - 1) / kCtaKeys), (unsigned)Hkv, (unsigned)b->n_req);
  score_mma_partial_kernel<<<grid, kMmaThreads, smem, sm>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k, b->cu_seqlens,
                                                            obs, H, Hkv, d, scale_log2, n_kb, rows_max, partial);
  PK_CUDA(cudaGetLastError());
  const int64_t n_lse = (int64_t)b->n_req * H * obs;
  score_lse_merge_kernel<<<(unsigned)((n_lse + 255) / 256), 256, 0, sm>>>(partial, b->cu_seqlens, obs, H, Hkv, n_kb,
                                                                         rows_max, b->n_req, lse2);
  PK_CUDA(cudaGetLastError());
  score_mma_colsum_kernel<<<grid, kMmaThreads, smem, sm>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k, b->cu_seqlens,
                                                           window, obs, H, Hkv, d, scale_log2, lse2, b->total_tokens, c_out);
  PK_CUDA(cudaGetLastError());
  return PUREKV_OK;
}

template <typename T>
static purekv_status launch_score(const void* q, const void* k, float* c_out, const purekv_batch* b, int32_t window,
                                  int32_t obs, int32_t H, int32_t Hkv, int32_t d, float scale, float* lse2,
                                  cudaStream_t sm) {
  const int32_t ml = max_len(b);
  const int32_t w = std::min(obs, ml);  // accumulated rows per head: the row blocks of the first pass
  const int32_t G = H / Hkv;
  const size_t smem = (size_t)(kRB + kKB) * (d + 4) * sizeof(float);
  {
    static std::atomic<uint64_t> smem_allowed{0};
    const purekv_status st_smem = allow_max_dynamic_smem(score_lse_kernel<T>, smem_allowed);
    if (st_smem != PUREKV_OK) return st_smem;
  }
  {
    static std::atomic<uint64_t> smem_allowed{0};
    const purekv_status st_smem = allow_max_dynamic_smem(score_colsum_kernel<T>, smem_allowed);
    if (st_smem != PUREKV_OK) return st_smem;
  }
  const float scale_log2 = scale * 1.4426950408889634f;
  dim3 g1((unsigned)((G * w + kRB - 1) / kRB), (unsigned)Hkv, (unsigned)b->n_req);
  score_lse_kernel<T><<<g1, kThreads, smem, sm>>>((const T*)q, (const T*)k, b->cu_seqlens, obs, H, Hkv, d, scale_log2,
                                                  lse2);
  PK_CUDA(cudaGetLastError());
  dim3 g2((unsigned)((ml + kKB - 1) / kKB), (unsigned)Hkv, (unsigned)b->n_req);
  score_colsum_kernel<T><<<g2, kThreads, smem, sm>>>((const T*)q, (const T*)k, b->cu_seqlens, window, obs, H, Hkv, d,
                                                     scale_log2, lse2, b->total_tokens, c_out);
  PK_CUDA(cudaGetLastError());
  return PUREKV_OK;
}

// Average pooling of the scores along the key axis (the pooled observation window of App. A.1's policies): each
// non-recent key takes the mean over `pool` positions centred on it, positions outside the non-recent segment
// counting as zero.  grid (key blocks of 256 over the longest request, n_kv_heads, n_req).
__global__ void __launch_bounds__(256) score_pool_kernel(const float* __restrict__ c_in, const int32_t* __restrict__ cu_seqlens,
                                                         int32_t window, int32_t pool, int64_t n_tokens,
                                                         float* __restrict__ c_out) {
  const int32_t r = blockIdx.z, g = blockIdx.y, j = blockIdx.x * 256 + threadIdx.x;
  const int32_t base = cu_seqlens[r], len = cu_seqlens[r + 1] - base;
  if (j >= len) return;
  const int32_t nr = len - min(window, len), half = pool / 2;
  const float* in = c_in + (int64_t)g * n_tokens + base;
  float sum = 0.f;
  if (j < nr)
    for (int32_t jj = max(0, j - half); jj <= min(nr - 1, j + half); ++jj) sum += in[jj];
  c_out[(int64_t)g * n_tokens + base + j] = sum / (float)(2 * half + 1);
}

// the last `obs` rows of every request are accumulated; < 0 or beyond the longest request: all rows
static int32_t obs_stride(const purekv_batch* b, int32_t obs_rows) {
  const int32_t ml = std::max(max_len(b), 1);
  return (obs_rows < 0 || obs_rows > ml) ? ml : std::max(obs_rows, 1);
}

// floats of log-sum-exp values per (request, head, accumulated row), plus (max, sum) pairs per 64-key block for
// the tensor-core path
static size_t score_ws_floats(const purekv_batch* batch, int32_t obs, int32_t n_q_heads) {
  const size_t rows = (size_t)batch->n_req * n_q_heads * (size_t)std::max(obs, 1);
  const size_t n_kb = ((size_t)max_len(batch) + kMmaKeys - 1) / kMmaKeys;
  return ((rows + 63) & ~(size_t)63) + rows * 2 * n_kb;
}

}  // namespace purekv

using namespace purekv;

extern "C" size_t purekv_score_ws_bytes(const purekv_batch* batch, int32_t window, int32_t n_q_heads) {
  if (!batch || window < 0 || n_q_heads < 0 || !batch->h_cu_seqlens) return 0;
  return score_ws_floats(batch, window, n_q_heads) * sizeof(float) + 256;
}

extern "C" size_t purekv_score_ex_ws_bytes(const purekv_batch* batch, int32_t obs_rows, int32_t pool, int32_t n_q_heads,
                                           int32_t n_kv_heads) {
  if (!batch || n_q_heads < 0 || n_kv_heads < 0 || !batch->h_cu_seqlens) return 0;
  size_t floats = score_ws_floats(batch, obs_stride(batch, obs_rows), n_q_heads);
  if (pool > 1) floats += (((size_t)n_kv_heads * batch->total_tokens) + 63) & ~(size_t)63;  // the scores before pooling
  return floats * sizeof(float) + 256;
}

// Common body of the score entry points: `obs_rows` accumulated rows (Eq. 2: the window), then pooling.
static purekv_status score_impl(const char* who, const void* q, const void* k, float* c_out, const purekv_batch* batch,
                                int32_t window, int32_t obs_rows, int32_t pool, int32_t n_q_heads, int32_t n_kv_heads,
                                int32_t head_dim, purekv_dtype dtype, float softmax_scale, void* ws, size_t ws_bytes,
                                size_t ws_need, void* stream) {
  purekv_status st = check_batch(batch, true);
  if (st != PUREKV_OK) return st;
  if (batch->total_tokens == 0 || batch->n_req == 0) return PUREKV_OK;  // empty batch: nothing to do
  PK_REQUIRE(q && k && c_out, PUREKV_ERR_INVALID_ARG, "%s: null pointer", who);
  PK_REQUIRE(n_q_heads >= 1 && n_kv_heads >= 1 && n_q_heads % n_kv_heads == 0, PUREKV_ERR_INVALID_ARG,
             "n_q_heads %d must be a positive multiple of n_kv_heads %d", n_q_heads, n_kv_heads);
  PK_REQUIRE(window >= 1, PUREKV_ERR_INVALID_ARG, "window must be >= 1");
  PK_REQUIRE(pool >= 1 && pool % 2 == 1, PUREKV_ERR_INVALID_ARG, "pool %d must be odd and >= 1", pool);
  PK_REQUIRE(head_dim >= 4 && head_dim % 4 == 0 && head_dim <= 256, PUREKV_ERR_UNSUPPORTED,
             "head_dim %d: need a multiple of 4 up to 256", head_dim);
  PK_REQUIRE(dtype == PUREKV_BF16 || dtype == PUREKV_FP32, PUREKV_ERR_INVALID_ARG, "unknown dtype");
  PK_REQUIRE(n_kv_heads <= 65535 && batch->n_req <= 65535, PUREKV_ERR_UNSUPPORTED, "too many heads or requests");
  PK_REQUIRE(ws && ws_bytes >= ws_need, PUREKV_ERR_WORKSPACE, "%s: workspace of %zu bytes is too small (need %zu)", who,
             ws_bytes, ws_need);
  const int32_t obs = obs_stride(batch, obs_rows);
  float* lse2 = (float*)(((uintptr_t)ws + 255) & ~(uintptr_t)255);
  float* c_raw = pool > 1 ? lse2 + score_ws_floats(batch, obs, n_q_heads) : c_out;  // scores before pooling
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
  cudaStream_t sm = (cudaStream_t)stream;
  if (dtype == PUREKV_BF16 && head_dim % 16 == 0)
    st = launch_score_mma(q, k, c_raw, batch, window, obs, n_q_heads, n_kv_heads, head_dim, scale, lse2, sm);
  else if (dtype == PUREKV_BF16)
    st = launch_score<__nv_bfloat16>(q, k, c_raw, batch, window, obs, n_q_heads, n_kv_heads, head_dim, scale, lse2, sm);
  else
    st = launch_score<float>(q, k, c_raw, batch, window, obs, n_q_heads, n_kv_heads, head_dim, scale, lse2, sm);
  if (st != PUREKV_OK || pool == 1) return st;
  dim3 grid((unsigned)((max_len(batch) + 255) / 256), (unsigned)n_kv_heads, (unsigned)batch->n_req);
  score_pool_kernel<<<grid, 256, 0, sm>>>(c_raw, batch->cu_seqlens, window, pool, batch->total_tokens, c_out);
  PK_CUDA(cudaGetLastError());
  return PUREKV_OK;
}

extern "C" purekv_status purekv_lowlayer_score(const void* q, const void* k, float* c_out, const purekv_batch* batch,
                                               int32_t window, int32_t n_q_heads, int32_t n_kv_heads,
                                               int32_t head_dim, purekv_dtype dtype, float softmax_scale, void* ws,
                                               size_t ws_bytes, void* stream) {
  if (batch && batch->h_cu_seqlens && window >= 1 && n_q_heads >= 1)
    return score_impl("purekv_lowlayer_score", q, k, c_out, batch, window, window, 1, n_q_heads, n_kv_heads, head_dim, dtype,
                      softmax_scale, ws, ws_bytes, purekv_score_ws_bytes(batch, window, n_q_heads), stream);
  return score_impl("purekv_lowlayer_score", q, k, c_out, batch, window, window, 1, n_q_heads, n_kv_heads, head_dim, dtype,
                    softmax_scale, ws, ws_bytes, 0, stream);
}

extern "C" purekv_status purekv_lowlayer_score_ex(const void* q, const void* k, float* c_out, const purekv_batch* batch,
                                                  int32_t window, int32_t obs_rows, int32_t pool, int32_t n_q_heads,
                                                  int32_t n_kv_heads, int32_t head_dim, purekv_dtype dtype,
                                                  float softmax_scale, void* ws, size_t ws_bytes, void* stream) {
  const size_t need = (batch && batch->h_cu_seqlens && n_q_heads >= 1 && n_kv_heads >= 1)
                          ? purekv_score_ex_ws_bytes(batch, obs_rows, pool, n_q_heads, n_kv_heads) : 0;
  return score_impl("purekv_lowlayer_score_ex", q, k, c_out, batch, window, obs_rows, pool, n_q_heads, n_kv_heads, head_dim,
                    dtype, softmax_scale, ws, ws_bytes, need, stream);
}

// Device address of the static scratch array on the current device; resolved on the first call per device.
static purekv_status noalloc_scratch(float** out) {
  constexpr int kMaxDevices = 64;
  static std::mutex mu;
  static float* ptrs[kMaxDevices] = {};
  int dev = -1;
  PK_CUDA(cudaGetDevice(&dev));
  PK_REQUIRE(dev >= 0 && dev < kMaxDevices, PUREKV_ERR_UNSUPPORTED, "device ordinal %d is beyond %d", dev, kMaxDevices);
  std::lock_guard<std::mutex> lock(mu);
  if (!ptrs[dev]) {
    float* p = nullptr;
    PK_CUDA(cudaGetSymbolAddress((void**)&p, g_noalloc_score_scratch));
    PK_REQUIRE(p != nullptr, PUREKV_ERR_CUDA, "cudaGetSymbolAddress returned a null scratch address");
    ptrs[dev] = p;
  }
  *out = ptrs[dev];
  return PUREKV_OK;
}

extern "C" purekv_status purekv_lowlayer_score_noalloc(const void* q, const void* k, float* c_out,
                                                       const purekv_batch* batch, int32_t window, int32_t n_q_heads,
                                                       int32_t n_kv_heads, int32_t head_dim, purekv_dtype dtype,
                                                       float softmax_scale, void* stream) {
  purekv_status st = check_batch(batch, true);
  if (st != PUREKV_OK) return st;
  if (batch->total_tokens == 0 || batch->n_req == 0) return PUREKV_OK;  // empty batch: nothing to do
  PK_REQUIRE(window >= 1 && n_q_heads >= 1, PUREKV_ERR_INVALID_ARG, "window and n_q_heads must be >= 1");
  const size_t need = (purekv_score_ws_bytes(batch, window, n_q_heads) - 256) / sizeof(float);
  PK_REQUIRE(need <= kNoallocScoreFloats, PUREKV_ERR_WORKSPACE,
             "purekv_lowlayer_score_noalloc: this problem needs %zu scratch values, the built-in scratch holds %zu; "
             "use purekv_lowlayer_score with a caller-provided workspace",
             need, kNoallocScoreFloats);
  float* scratch = nullptr;
  if ((st = noalloc_scratch(&scratch)) != PUREKV_OK) return st;
  // The scratch needs no clearing: every entry that a later kernel of the call reads is written earlier in the call.
  return purekv_lowlayer_score(q, k, c_out, batch, window, n_q_heads, n_kv_heads, head_dim, dtype, softmax_scale,
                               scratch, (kNoallocScoreFloats + 64) * sizeof(float), stream);
}
