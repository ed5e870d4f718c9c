// purekv_decode_attention: one decoding step over the compacted cache of one layer (Sec. 3.1: later tokens attend
// to the compressed cache; the stage Table 3 times as decode latency).  Every request brings one new query per head;
// query head hq reads KV head hq / G of the request's kept rows.
//
// Split-KV, HBM bound: a CTA owns a chunk of one (request, KV head)'s kept keys and serves all G query heads of the
// group from one read of K and one of V.  bf16 runs on tensor cores (decode_tc_kernel, further down); the kernel
// described next serves fp32.  Rows are 256 bytes (bf16 d = 128 or fp32 d = 64): a half-warp covers a
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
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // the merge kernel may be placed meanwhile
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

// ---- bf16, d = 128 on tensor cores ---------------------------------------------------------------------------
// The CUDA-core kernel above spends about 100 instructions per key at G = 8; with mma.sync the group's heads are
// the 16 rows of an m16n8k16 tile and the arithmetic all but disappears beside the loads.  A warp takes 16 keys per
// trip: S = Q K^T as two n8 tiles (8 k-steps each), online softmax on the accumulator registers, which then serve
// unchanged as the A operand of O += P V (16 n8 tiles over d).  No shared-memory staging and no transposes: a dot
// product does not care in which order its terms are taken, so each thread feeds the k (and n) slots of the
// fragments from contiguous bytes of a row and the same order is used for the other operand --
//   Q K^T: thread (row lane/4, t = lane%4) holds d = 32t .. 32t+31 of its Q rows and of its key's K row;
//          k-step ks takes elements 4ks, 4ks+1 (k slots 2t, 2t+1) and 4ks+2, 4ks+3 (k slots 2t+8, 2t+9);
//   P V:   thread (g8 = lane/4, t) holds d = 16 g8 .. 16 g8+15 of the V rows of keys 2t, 2t+1, 8+2t, 9+2t of the trip;
//          n tile nt covers d = 16 j + nt (j = 0 .. 7), two keys' values paired per register by a byte permute.
__device__ __forceinline__ uint4 ldg16_stream(const uint4* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}
__device__ __forceinline__ void dec_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t dec_pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

constexpr float kDecRescale = 8.f;  // the reference maximum of a row moves only when a logit exceeds it by this (log2)

// grid (n_splits, H_kv, n_req), 128 threads; G <= 16.  Same outputs as decode_partial_kernel.
__global__ void __launch_bounds__(kDecThreads) decode_tc_kernel(
    const uint4* __restrict__ q, const uint4* __restrict__ kc, const uint4* __restrict__ vc,
    const int32_t* __restrict__ cu_kept, int32_t n_q_heads, int32_t n_kv_heads, int32_t chunk, float scale_log2,
    __nv_bfloat16* __restrict__ o, float* __restrict__ lse, float* __restrict__ part, int32_t n_splits) {
  constexpr int D = 128;
  // a row's 128 columns as four runs of 32 padded to 33, rows 132 apart: the 32 lanes of a store (8 rows x 4 runs)
  // fall into 32 different banks
  __shared__ float s_o[kDecThreads / 32][16][4 * 33];
  __shared__ float s_ml[kDecThreads / 32][16][2];

  const int32_t sp = blockIdx.x, g = blockIdx.y, r = blockIdx.z;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // the merge kernel may be placed meanwhile
  const int32_t G = n_q_heads / n_kv_heads;
  const int32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g8 = lane >> 2, t = lane & 3;
  const int64_t j0 = (int64_t)cu_kept[r] + (int64_t)sp * chunk;
  const int32_t n = (int32_t)max((int64_t)0, min((int64_t)cu_kept[r + 1], j0 + chunk) - j0);

  // A fragments of Q: rows g8 and g8 + 8 (heads of the group; rows past G are zero)
  uint32_t qa[8][4];
  {
    uint4 lo[4], hi[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      lo[c] = g8 < G ? __ldg(q + ((int64_t)r * n_q_heads + g * G + g8) * 16 + t * 4 + c) : make_uint4(0, 0, 0, 0);
      hi[c] = g8 + 8 < G ? __ldg(q + ((int64_t)r * n_q_heads + g * G + g8 + 8) * 16 + t * 4 + c) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      qa[2 * c][0] = lo[c].x; qa[2 * c][1] = hi[c].x; qa[2 * c][2] = lo[c].y; qa[2 * c][3] = hi[c].y;
      qa[2 * c + 1][0] = lo[c].z; qa[2 * c + 1][1] = hi[c].z; qa[2 * c + 1][2] = lo[c].w; qa[2 * c + 1][3] = hi[c].w;
    }
  }

  float oacc[16][4];
#pragma unroll
  for (int nt = 0; nt < 16; ++nt)
#pragma unroll
    for (int x = 0; x < 4; ++x) oacc[nt][x] = 0.f;
  float m_ref[2] = {-INFINITY, -INFINITY}, l_part[2] = {0.f, 0.f};  // rows g8 and g8 + 8

  for (int32_t k0 = warp * 16; k0 < n; k0 += (kDecThreads / 32) * 16) {
    // every load of the trip is requested before the first use; rows past the end repeat the last one (weight 0)
    uint4 kr[2][4], vr[4][2];
#pragma unroll
    for (int tl = 0; tl < 2; ++tl) {
      const uint4* row = kc + ((j0 + min(k0 + 8 * tl + g8, n - 1)) * n_kv_heads + g) * 16 + t * 4;
#pragma unroll
      for (int c = 0; c < 4; ++c) kr[tl][c] = ldg16_stream(row + c);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {  // keys 2t, 2t+1, 8+2t, 9+2t of the trip
      const int32_t key = k0 + (i >> 1) * 8 + 2 * t + (i & 1);
      const uint4* row = vc + ((j0 + min(key, n - 1)) * n_kv_heads + g) * 16 + g8 * 2;
      vr[i][0] = ldg16_stream(row);
      vr[i][1] = ldg16_stream(row + 1);
    }
    // S for the two tiles of 8 keys
    float sc[2][4];
#pragma unroll
    for (int tl = 0; tl < 2; ++tl) {
#pragma unroll
      for (int x = 0; x < 4; ++x) sc[tl][x] = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        dec_mma(sc[tl], qa[2 * c], kr[tl][c].x, kr[tl][c].y);
        dec_mma(sc[tl], qa[2 * c + 1], kr[tl][c].z, kr[tl][c].w);
      }
    }
    // log2 units; keys past the end weigh nothing.  sc[tl][0..1]: row g8, keys 2t, 2t+1 of tile tl; [2..3]: row g8 + 8
#pragma unroll
    for (int tl = 0; tl < 2; ++tl)
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int32_t key = k0 + 8 * tl + 2 * t + (x & 1);
        sc[tl][x] = key < n ? sc[tl][x] * scale_log2 : -INFINITY;
      }
    uint32_t pa[4];
#pragma unroll
    for (int rw = 0; rw < 2; ++rw) {
      float mx = fmaxf(fmaxf(sc[0][2 * rw], sc[0][2 * rw + 1]), fmaxf(sc[1][2 * rw], sc[1][2 * rw + 1]));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      if (mx > m_ref[rw] + kDecRescale) {  // the same for the four threads of the row
        const float alpha = m_ref[rw] == -INFINITY ? 0.f : dec_ex2(m_ref[rw] - mx);
        l_part[rw] *= alpha;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
          oacc[nt][2 * rw] *= alpha;
          oacc[nt][2 * rw + 1] *= alpha;
        }
        m_ref[rw] = mx;
      }
      const float p00 = dec_ex2(sc[0][2 * rw] - m_ref[rw]), p01 = dec_ex2(sc[0][2 * rw + 1] - m_ref[rw]);
      const float p10 = dec_ex2(sc[1][2 * rw] - m_ref[rw]), p11 = dec_ex2(sc[1][2 * rw + 1] - m_ref[rw]);
      l_part[rw] += (p00 + p01) + (p10 + p11);
      pa[rw] = dec_pack_bf16(p00, p01);      // k slots 2t, 2t+1: keys 2t, 2t+1 of tile 0
      pa[2 + rw] = dec_pack_bf16(p10, p11);  // k slots 2t+8, 2t+9: the same keys of tile 1
    }
    // O += P V
    const uint32_t* x0 = reinterpret_cast<const uint32_t*>(vr[0]);
    const uint32_t* y0 = reinterpret_cast<const uint32_t*>(vr[1]);
    const uint32_t* x1 = reinterpret_cast<const uint32_t*>(vr[2]);
    const uint32_t* y1 = reinterpret_cast<const uint32_t*>(vr[3]);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      dec_mma(oacc[2 * j], pa, __byte_perm(x0[j], y0[j], 0x5410), __byte_perm(x1[j], y1[j], 0x5410));
      dec_mma(oacc[2 * j + 1], pa, __byte_perm(x0[j], y0[j], 0x7632), __byte_perm(x1[j], y1[j], 0x7632));
    }
  }
  // a row's sum over its four threads; then the warps' results side by side in shared memory
#pragma unroll
  for (int rw = 0; rw < 2; ++rw) {
    l_part[rw] += __shfl_xor_sync(0xffffffffu, l_part[rw], 1);
    l_part[rw] += __shfl_xor_sync(0xffffffffu, l_part[rw], 2);
  }
#pragma unroll
  for (int nt = 0; nt < 16; ++nt)
#pragma unroll
    for (int x = 0; x < 4; ++x) s_o[warp][g8 + 8 * (x >> 1)][t * 33 + (x & 1) * 16 + nt] = oacc[nt][x];  // d = 32t + 16(x&1) + nt
  if (t == 0) {
    s_ml[warp][g8][0] = m_ref[0];
    s_ml[warp][g8][1] = l_part[0];
    s_ml[warp][g8 + 8][0] = m_ref[1];
    s_ml[warp][g8 + 8][1] = l_part[1];
  }
  __syncthreads();
  for (int32_t x = tid; x < G * D; x += kDecThreads) {
    const int32_t h = x / D, c = x % D;
    float m_all = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecThreads / 32; ++w)
      if (s_ml[w][h][1] > 0.f) m_all = fmaxf(m_all, s_ml[w][h][0]);
    float a = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < kDecThreads / 32; ++w)
      if (s_ml[w][h][1] > 0.f) {
        const float wgt = dec_ex2(s_ml[w][h][0] - m_all);
        a = fmaf(wgt, s_o[w][h][(c >> 5) * 33 + (c & 31)], a);
        l = fmaf(wgt, s_ml[w][h][1], l);
      }
    const int32_t hq = g * G + h;
    if (n_splits == 1) {
      o[((int64_t)r * n_q_heads + hq) * D + c] = __float2bfloat16(l > 0.f ? a / l : 0.f);
      if (c == 0 && lse) lse[(int64_t)r * n_q_heads + hq] = l > 0.f ? (m_all + log2f(l)) * 0.6931471805599453f : -INFINITY;
    } else {
      float* dst = part + (((int64_t)r * n_q_heads + hq) * n_splits + sp) * (D + 2);
      dst[c] = a;
      if (c == 0) {
        dst[D] = m_all;
        dst[D + 1] = l;
      }
    }
  }
}

// grid (H, n_req), D threads (D = 64 or 128): merges the chunks' partial results of one (request, head).  The
// chunks' weights 2^(m_s - m) are formed once, 128 chunks at a time, in shared memory; thread c then sums column c
// with independent loads.
template <typename T>
__global__ void decode_merge_kernel(const float* __restrict__ part, int32_t n_q_heads, int32_t n_splits, int32_t D,
                                    T* __restrict__ o, float* __restrict__ lse) {
  __shared__ float s_w[128];
  __shared__ float s_red[4];
  __shared__ float s_m;
  const int32_t hq = blockIdx.x, r = blockIdx.y, c = threadIdx.x, lane = c & 31, warp = c >> 5;
  const int32_t n_warps = (int32_t)blockDim.x >> 5;
  // launched with programmatic stream serialization: placed while the chunk kernel still runs, its partial results
  // are complete and visible from here on
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const float* src = part + ((int64_t)r * n_q_heads + hq) * n_splits * (D + 2);
  // the largest chunk maximum among chunks that hold anything
  float m = -INFINITY;
  for (int32_t s = c; s < n_splits; s += (int32_t)blockDim.x)
    if (src[(int64_t)s * (D + 2) + D + 1] > 0.f) m = fmaxf(m, src[(int64_t)s * (D + 2) + D]);
#pragma unroll
  for (int mask = 16; mask >= 1; mask >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, mask));
  if (lane == 0) s_red[warp] = m;
  __syncthreads();
  if (c == 0) {
    float mm = s_red[0];
    for (int32_t w = 1; w < n_warps; ++w) mm = fmaxf(mm, s_red[w]);
    s_m = mm;
  }
  __syncthreads();
  const float m_all = s_m;
  float a = 0.f, l = 0.f;
  for (int32_t s0 = 0; s0 < n_splits; s0 += 128) {
    const int32_t ns = min(128, n_splits - s0);
    __syncthreads();
    for (int32_t i = c; i < ns; i += (int32_t)blockDim.x) {
      const float ls = src[(int64_t)(s0 + i) * (D + 2) + D + 1];
      const float wgt = ls > 0.f ? dec_ex2(src[(int64_t)(s0 + i) * (D + 2) + D] - m_all) : 0.f;
      s_w[i] = wgt;
      l = fmaf(wgt, ls, l);  // this thread's share of the row sum
    }
    __syncthreads();
    const float* col = src + (int64_t)s0 * (D + 2) + c;
    int32_t i = 0;
    for (; i + 4 <= ns; i += 4) {
      const float v0 = col[(int64_t)i * (D + 2)], v1 = col[(int64_t)(i + 1) * (D + 2)];
      const float v2 = col[(int64_t)(i + 2) * (D + 2)], v3 = col[(int64_t)(i + 3) * (D + 2)];
      a = fmaf(s_w[i], v0, a); a = fmaf(s_w[i + 1], v1, a); a = fmaf(s_w[i + 2], v2, a); a = fmaf(s_w[i + 3], v3, a);
    }
    for (; i < ns; ++i) a = fmaf(s_w[i], col[(int64_t)i * (D + 2)], a);
  }
#pragma unroll
  for (int mask = 16; mask >= 1; mask >>= 1) l += __shfl_xor_sync(0xffffffffu, l, mask);
  __syncthreads();
  if (lane == 0) s_red[warp] = l;
  __syncthreads();
  l = 0.f;
  for (int32_t w = 0; w < n_warps; ++w) l += s_red[w];
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
  PK_REQUIRE(G <= (dtype == PUREKV_BF16 ? 16 : 8), PUREKV_ERR_UNSUPPORTED,
             "purekv_decode_attention: at most 16 (bf16) or 8 (fp32) query heads per KV head");
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
    decode_tc_kernel<<<grid, kDecThreads, 0, sm>>>((const uint4*)q, (const uint4*)k_cache, (const uint4*)v_cache, cu_kept,
                                                  n_q_heads, n_kv_heads, chunk, scale_log2, (__nv_bfloat16*)o, lse, part,
                                                  n_splits);
  } else {
    PK_DECODE(float)
  }
#undef PK_DECODE
  PK_CUDA(cudaGetLastError());
  if (n_splits > 1) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_q_heads, (unsigned)n_req);
    cfg.blockDim = dim3((unsigned)head_dim);
    cfg.stream = sm;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see griddepcontrol in the kernels
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float* part_c = part;
    if (dtype == PUREKV_BF16)
      PK_CUDA(cudaLaunchKernelEx(&cfg, decode_merge_kernel<__nv_bfloat16>, part_c, n_q_heads, n_splits, head_dim,
                                 (__nv_bfloat16*)o, lse));
    else
      PK_CUDA(cudaLaunchKernelEx(&cfg, decode_merge_kernel<float>, part_c, n_q_heads, n_splits, head_dim, (float*)o, lse));
    PK_CUDA(cudaGetLastError());
  }
  return PUREKV_OK;
}

}  // extern "C"
