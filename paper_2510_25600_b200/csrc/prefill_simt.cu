// CUDA-core ST-SpAttn prefill (Sec. 3.2) for the shapes the tensor-core kernel does not take:
// fp32 inputs (computed in fp32 throughout) and bf16 with head_dim other than 128.
//
// One CTA = one query tile (<= 64 rows) of one query head, walking the plan's list of kept key
// tiles (general tiles carry a bit mask in the plan).  K and V tiles are staged in shared memory as fp32.  A warp owns rows warp, warp+4, ...
// of the tile; for a row the lanes split the keys of the tile for q.k, the row's online-softmax
// state (max, sum, d/32 output values per lane) lives in registers, and probabilities pass
// through a per-warp shared buffer for the P.V product where the lanes split the head dim.
#include "common.cuh"
#include "prefill.cuh"

namespace purekv {

constexpr int kSimtThreads = 128;
constexpr int kSimtWarps = 4;
constexpr int kMaxRowsPerWarp = 16;  // tile_q <= 64

template <typename T, int DPL>  // head_dim = 32 * DPL
__global__ void __launch_bounds__(kSimtThreads) prefill_simt_kernel(
    const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, T* __restrict__ o,
    float* __restrict__ lse, const uint8_t* __restrict__ plan, int32_t n_q_heads, int32_t n_kv_heads,
    float scale_log2) {
  constexpr int D = 32 * DPL;
  constexpr int LD = D + 1;
  extern __shared__ __align__(16) float smem[];
  const PlanHeader* hdr = reinterpret_cast<const PlanHeader*>(plan);
  const QTile* qtiles = reinterpret_cast<const QTile*>(plan + hdr->off_qtiles);
  const int32_t* order = reinterpret_cast<const int32_t*>(plan + hdr->off_order);
  const int2* entries = reinterpret_cast<const int2*>(plan + hdr->off_entries);
  const uint32_t* masks = reinterpret_cast<const uint32_t*>(plan + hdr->off_masks);
  const int32_t tq = hdr->tile_q, tk = hdr->tile_k, wpr = hdr->words_per_row;
  const QTile qt = qtiles[order[blockIdx.x]];
  const int32_t hq = blockIdx.y, g = hq / (n_q_heads / n_kv_heads);
  const int32_t q_rel0 = qt.q_start - qt.req_start;

  float* qs = smem;                         // [tq][D]
  float* ks = qs + tq * D;                  // [tk][LD]
  float* vs = ks + tk * LD;                 // [tk][LD]
  float* ps = vs + tk * LD;                 // [warps][tk]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int x = tid; x < tq * D; x += kSimtThreads) {
    const int row = x / D, c = x % D;
    qs[x] = row < qt.q_rows ? to_f32(q[((int64_t)(qt.q_start + row) * n_q_heads + hq) * D + c]) : 0.f;
  }

  float m[kMaxRowsPerWarp], l[kMaxRowsPerWarp], acc[kMaxRowsPerWarp][DPL];
#pragma unroll
  for (int rr = 0; rr < kMaxRowsPerWarp; ++rr) {
    m[rr] = -INFINITY;
    l[rr] = 0.f;
#pragma unroll
    for (int c = 0; c < DPL; ++c) acc[rr][c] = 0.f;
  }

  for (int32_t e = 0; e < qt.entry_count; ++e) {
    const int2 ent = entries[qt.entry_begin + e];
    const int32_t cls = ent.x & 3, j0 = (ent.x >> 4) * tk;
    __syncthreads();
    for (int x = tid; x < tk * D; x += kSimtThreads) {
      const int row = x / D, c = x % D;
      const bool in = j0 + row < qt.req_len;
      const int64_t src = ((int64_t)(qt.req_start + j0 + row) * n_kv_heads + g) * D + c;
      ks[row * LD + c] = in ? to_f32(k[src]) : 0.f;
      vs[row * LD + c] = in ? to_f32(v[src]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int rr = 0; rr < kMaxRowsPerWarp; ++rr) {
      const int row = warp + kSimtWarps * rr;
      if (row >= qt.q_rows) continue;  // warp-uniform
      const int32_t i = q_rel0 + row;
      const float* qrow = qs + row * D;
      float tmax = -INFINITY;
      float sv[4];  // tk <= 128 -> at most 4 keys per lane
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const int c = lane + 32 * kk;
        sv[kk] = -INFINITY;
        if (c < tk) {
          bool keep = cls == kTileFull || j0 + c <= i;
          if (cls == kTileGeneral) keep = (__ldg(masks + ent.y + row * wpr + (c >> 5)) >> (c & 31)) & 1u;
          if (keep) {
            float s = 0.f;
            const float* krow = ks + c * LD;
#pragma unroll 8
            for (int dd = 0; dd < D; ++dd) s = fmaf(qrow[dd], krow[dd], s);
            sv[kk] = s * scale_log2;
            tmax = fmaxf(tmax, sv[kk]);
          }
        }
      }
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, off));
      if (tmax == -INFINITY) continue;  // no kept key for this row in this tile (warp-uniform)
      const float mn = fmaxf(m[rr], tmax);
      const float alpha = exp2f(m[rr] - mn);  // 0 when m was -inf
      float psum = 0.f;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const int c = lane + 32 * kk;
        if (c < tk) {
          const float p = exp2f(sv[kk] - mn);  // exp2(-inf) = 0 for masked keys
          ps[warp * tk + c] = p;
          psum += p;
        }
      }
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, off);
      l[rr] = l[rr] * alpha + psum;
      m[rr] = mn;
      __syncwarp();
#pragma unroll
      for (int c = 0; c < DPL; ++c) acc[rr][c] *= alpha;
      for (int kc = 0; kc < tk; ++kc) {
        const float p = ps[warp * tk + kc];
#pragma unroll
        for (int c = 0; c < DPL; ++c) acc[rr][c] = fmaf(p, vs[kc * LD + lane + 32 * c], acc[rr][c]);
      }
      __syncwarp();
    }
  }
#pragma unroll
  for (int rr = 0; rr < kMaxRowsPerWarp; ++rr) {
    const int row = warp + kSimtWarps * rr;
    if (row >= qt.q_rows) continue;
    const float inv = 1.f / l[rr];
    T* dst = o + ((int64_t)(qt.q_start + row) * n_q_heads + hq) * D;
#pragma unroll
    for (int c = 0; c < DPL; ++c) {
      const float val = acc[rr][c] * inv;
      if constexpr (sizeof(T) == 2) dst[lane + 32 * c] = __float2bfloat16_rn(val);
      else dst[lane + 32 * c] = val;
    }
    if (lse && lane == 0)
      lse[(int64_t)hq * hdr->total_tokens + qt.q_start + row] = (m[rr] + log2f(l[rr])) * 0.6931471805599453f;
  }
}

template <typename T, int DPL>
static purekv_status launch(const PrefillArgs& a) {
  const int D = 32 * DPL;
  const size_t smem = ((size_t)a.info->tile_q * D + 2 * (size_t)a.info->tile_k * (D + 1) +
                       (size_t)kSimtWarps * a.info->tile_k) * sizeof(float);
  PK_REQUIRE(smem <= 227 * 1024, PUREKV_ERR_UNSUPPORTED,
             "head_dim %d with tile %d needs %zu bytes of shared memory", D, a.info->tile_k, smem);
  {
    static std::atomic<uint64_t> smem_allowed{0};
    const purekv_status st_smem = allow_max_dynamic_smem(prefill_simt_kernel<T, DPL>, smem_allowed);
    if (st_smem != PUREKV_OK) return st_smem;
  }
  dim3 grid((unsigned)a.info->n_qtiles, (unsigned)a.n_q_heads);
  prefill_simt_kernel<T, DPL><<<grid, kSimtThreads, smem, a.stream>>>(
      (const T*)a.q, (const T*)a.k, (const T*)a.v, (T*)a.o, a.lse, (const uint8_t*)a.plan, a.n_q_heads, a.n_kv_heads,
      a.scale * 1.4426950408889634f);
  PK_CUDA(cudaGetLastError());
  return PUREKV_OK;
}

purekv_status launch_prefill_simt(const PrefillArgs& a) {
  PK_REQUIRE(a.info->tile_q <= 64 && a.info->tile_q >= 1 && a.info->tile_k <= 128, PUREKV_ERR_UNSUPPORTED,
             "CUDA-core prefill needs a plan with tile_q <= 64");
  const bool bf = a.dtype == PUREKV_BF16;
  switch (a.head_dim) {
    case 32: return bf ? launch<__nv_bfloat16, 1>(a) : launch<float, 1>(a);
    case 64: return bf ? launch<__nv_bfloat16, 2>(a) : launch<float, 2>(a);
    case 128: return bf ? launch<__nv_bfloat16, 4>(a) : launch<float, 4>(a);
    case 256: return bf ? launch<__nv_bfloat16, 8>(a) : launch<float, 8>(a);
    default: break;
  }
  set_error("head_dim %d has no prefill kernel (supported: 32, 64, 128, 256)", a.head_dim);
  return PUREKV_ERR_UNSUPPORTED;
}

}  // namespace purekv
