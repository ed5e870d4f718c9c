// Tensor-core ST-SpAttn prefill (Sec. 3.2) for bf16, head_dim 128, on sm_100a.
//
// One CTA = one 128-row query tile of a PAIR of query heads that share a KV head ("slots"), so
// every K/V tile staged in shared memory feeds two heads.  It walks the plan's list of kept key
// tiles: key blocks the mask removes are never read.  Roles:
//   warp 0      TMA producer: Q of both slots once, then K and V tiles (128B-swizzled, two
//               64-column panels each) into a ring of stages.
//   warp 1      owns the 512 TMEM columns; one lane issues tcgen05.mma, alternating slots:
//               S = Q K^T (K-major A and B from shared memory) and
//               O += P V (A = bf16 P from TMEM, B = V as MN-major shared-memory operand),
//               so the tensor pipe works on one slot while the other slot's rows are in softmax.
//   warps 2-9   one thread per query row of a slot: the row of S from TMEM into registers, the
//               tile's predicate class (full / causal / bit mask from the plan), online softmax in
//               the log2 domain with lazy rescaling of O, bf16 P written over S, final normalise
//               and store.
// Every wait on an mbarrier is bounded in time; on expiry the CTA raises a shared abort flag,
// sets the device status word, drains, frees TMEM and exits.
#include <cuda.h>

#include "prefill.cuh"

namespace purekv {
namespace tc {

constexpr int kD = 128;
constexpr int kBQ = 128;
constexpr int kThreads = 320;  // warp 0 TMA, warp 1 MMA, warps 2-5 softmax of slot 0, warps 6-9 of slot 1
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColO = 256;
constexpr uint64_t kWaitLimitNs = 1000ull * 1000ull * 1000ull;  // 1 s per wait
constexpr float kRescaleThreshold = 8.0f;                        // log2 units

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: false if the abort flag is up or the time limit passed (then raises the flag).
// The wall-clock timer is slow to read, so it is consulted only every 1024 failed polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  uint64_t t0 = 0;
  uint32_t it = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++it & 1023u) == 0u) {
      if (*abort_flag) return false;
      const uint64_t now = global_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t c0, int32_t c1,
                                            int32_t c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

#define PK_R8(r, o) "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), "=r"(r[o + 6]), "=r"(r[o + 7])
#define PK_W8(r, o) "r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]), "r"(r[o + 6]), "r"(r[o + 7])

// 32 lanes x 32 consecutive columns -> 32 registers per thread (thread = lane = row).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : PK_R8(r, 0), PK_R8(r, 8), PK_R8(r, 16), PK_R8(r, 24)
      : "r"(taddr)
      : "memory");
}
// Same load into elements OFF .. OFF+31 of a larger register array.
template <int OFF, int N>
__device__ __forceinline__ void tmem_ld32_at(uint32_t taddr, uint32_t (&r)[N]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : PK_R8(r, OFF + 0), PK_R8(r, OFF + 8), PK_R8(r, OFF + 16), PK_R8(r, OFF + 24)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};" ::PK_W8(r, 0),
      PK_W8(r, 8), PK_W8(r, 16), PK_W8(r, 24), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};" ::PK_W8(r, 0),
      PK_W8(r, 8), "r"(taddr)
      : "memory");
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor for kind::f16: bf16 x bf16 -> fp32, M = 128.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(128 >> 4) << 24);
}

template <int BK>
struct Cfg {
  static constexpr int kStages = BK == 64 ? 4 : 2;  // K/V ring depth (32 KB resp. 64 KB per stage)
  static constexpr int kSBuf = BK == 64 ? 2 : 1;    // S buffers per slot: kSBuf * BK = 128 TMEM columns
};

template <int BK>
struct __align__(8) Barriers {
  static constexpr int ST = Cfg<BK>::kStages, SB = Cfg<BK>::kSBuf;
  uint64_t q_full;
  uint64_t k_full[ST], k_empty[ST], v_full[ST], v_empty[ST];
  uint64_t s_full[2][SB];  // MMA -> softmax: S of (slot, buffer) is complete
  uint64_t p_full[2][SB];  // softmax -> MMA: P written (and O rescaled) by all 128 row threads
  uint64_t o_done[2];      // one completion per P.V product of the slot
  uint64_t o_final[2];     // completes once, after the slot's last P.V product
  uint64_t drain;
};

// TMEM columns: S(slot, buf) at slot*128 + buf*BK (P aliases its first BK/2 columns), O(slot) at 256 + slot*128.
template <int BK>
__global__ void __launch_bounds__(kThreads, 1) prefill_tc_kernel(
    const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
    const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ o, float* __restrict__ lse,
    const uint8_t* __restrict__ plan, int32_t n_q_heads, int32_t n_kv_heads, float scale_log2,
    int32_t* __restrict__ status) {
  constexpr int ST = Cfg<BK>::kStages, SB = Cfg<BK>::kSBuf;
  constexpr uint32_t kPanelQ = kBQ * 128;  // bytes of one 64-column panel of a Q tile
  constexpr uint32_t kTileQ = 2 * kPanelQ;
  constexpr uint32_t kPanelKV = BK * 128;  // bytes of one 64-column panel of a K or V tile
  constexpr uint32_t kTileKV = 2 * kPanelKV;
  extern __shared__ uint8_t smem_raw[];
  __shared__ Barriers<BK> bars;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;

  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = smem0;                 // [2 slots][2 panels][128 rows x 128 B]
  const uint32_t sK = sQ + 2 * kTileQ;       // [ST][2 panels][BK rows x 128 B]
  const uint32_t sV = sK + ST * kTileKV;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const PlanHeader* hdr = reinterpret_cast<const PlanHeader*>(plan);
  const QTile* qtiles = reinterpret_cast<const QTile*>(plan + hdr->off_qtiles);
  const int32_t* order = reinterpret_cast<const int32_t*>(plan + hdr->off_order);
  const int2* entries = reinterpret_cast<const int2*>(plan + hdr->off_entries);
  const uint32_t* masks = reinterpret_cast<const uint32_t*>(plan + hdr->off_masks);
  // blockIdx.x = rank of the query tile in the longest-first order * n_pairs + pair, so the long lists of
  // every head start first.  A pair = (KV head, two of its query heads); the last pair of an odd group is single.
  const int32_t G = n_q_heads / n_kv_heads, ppg = (G + 1) >> 1, n_pairs = n_kv_heads * ppg;
  const QTile qt = qtiles[order[blockIdx.x / n_pairs]];
  const int32_t pair = blockIdx.x % n_pairs;
  const int32_t g = pair / ppg, pr = pair % ppg;
  const int32_t hq0 = g * G + 2 * pr;
  const int32_t n_slots = (2 * pr + 1 < G) ? 2 : 1;
  const int32_t nt = qt.entry_count;
  const int2* ent = entries + qt.entry_begin;
  volatile int* abort_flag = &abort_s;

  if (tid == 0) {
    abort_s = *reinterpret_cast<volatile int32_t*>(status) != 0;  // an earlier CTA already failed
    mbar_init(smem_u32(&bars.q_full), 1);
    for (int s = 0; s < ST; ++s) {
      mbar_init(smem_u32(&bars.k_full[s]), 1);
      mbar_init(smem_u32(&bars.k_empty[s]), 1);
      mbar_init(smem_u32(&bars.v_full[s]), 1);
      mbar_init(smem_u32(&bars.v_empty[s]), 1);
    }
    for (int sl = 0; sl < 2; ++sl) {
      for (int b = 0; b < SB; ++b) {
        mbar_init(smem_u32(&bars.s_full[sl][b]), 1);
        mbar_init(smem_u32(&bars.p_full[sl][b]), 128);
      }
      mbar_init(smem_u32(&bars.o_done[sl]), 1);
      mbar_init(smem_u32(&bars.o_final[sl]), 1);
    }
    mbar_init(smem_u32(&bars.drain), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_s), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  const bool start_ok = abort_s == 0;

  if (start_ok && warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      mbar_expect_tx(smem_u32(&bars.q_full), n_slots * kTileQ);
      for (int sl = 0; sl < n_slots; ++sl) {
        tma_load_3d(sQ + sl * kTileQ, &tm_q, smem_u32(&bars.q_full), 0, hq0 + sl, qt.q_start);
        tma_load_3d(sQ + sl * kTileQ + kPanelQ, &tm_q, smem_u32(&bars.q_full), 64, hq0 + sl, qt.q_start);
      }
      int32_t issued_k = 0, issued_v = 0;
      for (int32_t n = 0; n < nt; ++n) {
        const int32_t s = n % ST;
        const uint32_t par = ((n / ST) - 1) & 1;
        const int32_t tok = qt.req_start + (ent[n].x >> 2) * BK;
        if (n >= ST && !mbar_wait(smem_u32(&bars.k_empty[s]), par, abort_flag)) break;
        mbar_expect_tx(smem_u32(&bars.k_full[s]), kTileKV);
        tma_load_3d(sK + s * kTileKV, &tm_k, smem_u32(&bars.k_full[s]), 0, g, tok);
        tma_load_3d(sK + s * kTileKV + kPanelKV, &tm_k, smem_u32(&bars.k_full[s]), 64, g, tok);
        issued_k = n + 1;
        if (n >= ST && !mbar_wait(smem_u32(&bars.v_empty[s]), par, abort_flag)) break;
        mbar_expect_tx(smem_u32(&bars.v_full[s]), kTileKV);
        tma_load_3d(sV + s * kTileKV, &tm_v, smem_u32(&bars.v_full[s]), 0, g, tok);
        tma_load_3d(sV + s * kTileKV + kPanelKV, &tm_v, smem_u32(&bars.v_full[s]), 64, g, tok);
        issued_v = n + 1;
      }
      if (*abort_flag) {
        // drain: every issued copy must have landed before shared memory is released
        const uint64_t t0 = global_ns();
        for (int32_t n = max(0, issued_k - ST); n < issued_k; ++n)
          while (!mbar_try_wait(smem_u32(&bars.k_full[n % ST]), (n / ST) & 1) && global_ns() - t0 < kWaitLimitNs) {}
        for (int32_t n = max(0, issued_v - ST); n < issued_v; ++n)
          while (!mbar_try_wait(smem_u32(&bars.v_full[n % ST]), (n / ST) & 1) && global_ns() - t0 < kWaitLimitNs) {}
        while (!mbar_try_wait(smem_u32(&bars.q_full), 0) && global_ns() - t0 < kWaitLimitNs) {}
      }
    }
  } else if (start_ok && warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(BK, false);
      constexpr uint32_t idesc_pv = instr_desc(kD, true);
      // S(slot, n) = Q_slot K_n^T; the last slot to read K_n releases its stage
      auto issue_qk = [&](int32_t sl, int32_t n) -> bool {
        const int32_t s = n % ST, b = n % SB;
        if (!mbar_wait(smem_u32(&bars.k_full[s]), (n / ST) & 1, abort_flag)) return false;
        tc_fence_after();
        const uint32_t d_addr = tmem + sl * 128 + b * BK;
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
          const uint32_t qoff = sl * kTileQ + (ks >> 2) * kPanelQ + (ks & 3) * 32;
          const uint32_t koff = s * kTileKV + (ks >> 2) * kPanelKV + (ks & 3) * 32;
          mma_ss(d_addr, smem_desc(sQ + qoff, 16, 1024), smem_desc(sK + koff, 16, 1024), idesc_qk, ks > 0 ? 1u : 0u);
        }
        if (sl == n_slots - 1) tc_commit(smem_u32(&bars.k_empty[s]));
        tc_commit(smem_u32(&bars.s_full[sl][b]));
        return true;
      };
      // O(slot) += P(slot, n) V_n; the last slot to read V_n releases its stage
      auto issue_pv = [&](int32_t sl, int32_t n) -> bool {
        const int32_t s = n % ST, b = n % SB;
        if (!mbar_wait(smem_u32(&bars.v_full[s]), (n / ST) & 1, abort_flag)) return false;
        if (!mbar_wait(smem_u32(&bars.p_full[sl][b]), (n / SB) & 1, abort_flag)) return false;
        tc_fence_after();
        const uint32_t p_addr = tmem + sl * 128 + b * BK;
#pragma unroll
        for (int ks = 0; ks < BK / 16; ++ks) {
          // B = V tile, MN-major: 16 key rows (2 groups of 8, SBO 1024) x 128 dims (2 panels, LBO)
          const uint64_t bdesc = smem_desc(sV + s * kTileKV + ks * 2048, kPanelKV, 1024);
          mma_ts(tmem + kColO + sl * 128, p_addr + ks * 8, bdesc, idesc_pv, (n > 0 || ks > 0) ? 1u : 0u);
        }
        if (sl == n_slots - 1) tc_commit(smem_u32(&bars.v_empty[s]));
        tc_commit(smem_u32(&bars.o_done[sl]));
        if (n == nt - 1) tc_commit(smem_u32(&bars.o_final[sl]));
        return true;
      };
      bool ok = mbar_wait(smem_u32(&bars.q_full), 0, abort_flag);
      for (int32_t n = 0; ok && n < SB && n < nt; ++n)
        for (int32_t sl = 0; ok && sl < n_slots; ++sl) ok = issue_qk(sl, n);
      for (int32_t n = 0; ok && n < nt; ++n)
        for (int32_t sl = 0; ok && sl < n_slots; ++sl) {
          ok = issue_pv(sl, n);
          if (ok && n + SB < nt) ok = issue_qk(sl, n + SB);  // in order behind P.V of tile n, which frees S(slot, n % SB)
        }
      if (!ok) {
        // leaving early: let every issued MMA finish before TMEM is released
        tc_commit(smem_u32(&bars.drain));
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(smem_u32(&bars.drain), 0) && global_ns() - t0 < kWaitLimitNs) {}
      }
    }
  } else if (start_ok && (warp - 2) / 4 < n_slots) {
    // ---------------- softmax / epilogue: one thread per query row of one slot ----------------
    const int sl = (warp - 2) >> 2;
    const int quad = warp & 3;  // TMEM lane quadrant this warp may access
    const int row = quad * 32 + lane;
    const int32_t hq = hq0 + sl;
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16);
    const bool row_valid = row < qt.q_rows;
    const int32_t i_rel = qt.q_start - qt.req_start + row;
    const int32_t wpr = BK / 32;
    // waits are made warp-uniform: the TMEM loads/stores below need the whole warp
    auto wait_w = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag) ? 1 : 0) != 0;
    };
    float m_ref = -INFINITY, l_sum = 0.f;
    bool ok = true;
    for (int32_t n = 0; n < nt; ++n) {
      const int32_t b = n % SB;
      const int2 e = ent[n];
      const int32_t cls = e.x & 3, j0 = (e.x >> 2) * BK;
      uint32_t keep[BK / 32];
      if (cls == kTileGeneral) {  // this row's bits of the tile's mask (read before the wait to hide the latency)
        const uint32_t* mrow = masks + e.y + row * wpr;
#pragma unroll
        for (int c = 0; c < BK / 32; ++c) keep[c] = __ldg(mrow + c);
      } else if (cls == kTileDiag) {
        const int32_t n_ok = min(BK, max(0, i_rel - j0 + 1));  // causal: columns 0 .. n_ok-1
#pragma unroll
        for (int c = 0; c < BK / 32; ++c) {
          const int32_t k_in = min(32, max(0, n_ok - 32 * c));
          keep[c] = k_in >= 32 ? 0xFFFFFFFFu : ((1u << k_in) - 1u);
        }
      }
      if (!wait_w(smem_u32(&bars.s_full[sl][b]), (n / SB) & 1)) { ok = false; break; }
      tc_fence_after();
      const uint32_t s_addr = t_lane + sl * 128 + b * BK;
      // Row maximum.  BK = 64: the whole row of S stays in registers; BK = 128: the register file cannot hold
      // 128 values beside the rest (168 registers per thread at this CTA size), so the row is read twice.
      constexpr int NR = BK == 64 ? 64 : 32;
      uint32_t r[NR];
      float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      if constexpr (BK == 64) {
        tmem_ld32_at<0>(s_addr, r);
        tmem_ld32_at<32>(s_addr + 32, r);
        tc_wait_ld();
        if (cls != kTileFull) {
#pragma unroll
          for (int x = 0; x < 64; ++x)
            if (!((keep[x >> 5] >> (x & 31)) & 1u)) r[x] = 0xFF800000u;  // -inf: drops out of max and exp
        }
#pragma unroll
        for (int x = 0; x < 64; ++x) mx[x & 3] = fmaxf(mx[x & 3], __uint_as_float(r[x]));
      } else {
#pragma unroll
        for (int c = 0; c < BK / 32; ++c) {
          tmem_ld32_at<0>(s_addr + 32 * c, r);
          tc_wait_ld();
          if (cls != kTileFull) {
#pragma unroll
            for (int x = 0; x < 32; ++x)
              if (!((keep[c] >> x) & 1u)) r[x] = 0xFF800000u;
          }
#pragma unroll
          for (int x = 0; x < 32; ++x) mx[x & 3] = fmaxf(mx[x & 3], __uint_as_float(r[x]));
        }
      }
      const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale_log2;  // scale > 0
      // lazy rescale: move the reference only when the maximum grew by more than the threshold
      float m_use = m_ref;
      const bool grow = m_tile > m_ref + kRescaleThreshold || (m_ref == -INFINITY && m_tile > -INFINITY);
      if (grow) m_use = m_tile;
      const float m_sub = m_use == -INFINITY ? 0.f : m_use;
      // rescale O and the running sum where the reference moved (warp-uniform decision)
      const float alpha = grow ? (m_ref == -INFINITY ? 0.f : ex2(m_ref - m_use)) : 1.f;
      if (n > 0 && __any_sync(0xffffffffu, grow)) {
        // O must be quiescent: with one S buffer, S of tile n was issued behind P.V of tile n-1, so it is;
        // with two, S of tile n only implies P.V of tile n-2 (o_done is then in phase n-1 or n).
        if (SB > 1 && !wait_w(smem_u32(&bars.o_done[sl]), (n - 1) & 1)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < kD / 32; ++c) {
          uint32_t t[32];
          tmem_ld32(t_lane + kColO + sl * 128 + 32 * c, t);
          tc_wait_ld();
#pragma unroll
          for (int x = 0; x < 32; ++x) t[x] = __float_as_uint(__uint_as_float(t[x]) * alpha);
          tmem_st32(t_lane + kColO + sl * 128 + 32 * c, t);
        }
      }
      // probabilities -> bf16 P over the S columns, row sum in fp32
      float ls[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c = 0; c < BK / 32; ++c) {
        constexpr int kOff = BK == 64 ? 32 : 0;
        if constexpr (BK == 128) {
          tmem_ld32_at<0>(s_addr + 32 * c, r);
          tc_wait_ld();
          if (cls != kTileFull) {
#pragma unroll
            for (int x = 0; x < 32; ++x)
              if (!((keep[c] >> x) & 1u)) r[x] = 0xFF800000u;
          }
        }
        uint32_t pk[16];
#pragma unroll
        for (int x = 0; x < 32; x += 2) {
          const float p0 = ex2(fmaf(__uint_as_float(r[kOff * c + x]), scale_log2, -m_sub));
          const float p1 = ex2(fmaf(__uint_as_float(r[kOff * c + x + 1]), scale_log2, -m_sub));
          ls[(x >> 1) & 3] += p0 + p1;
          pk[x >> 1] = pack_bf16(p0, p1);
        }
        // P chunk c lands on S columns 16c..16c+15, which this thread has already consumed
        tmem_st16(s_addr + 16 * c, pk);
      }
      l_sum = l_sum * alpha + ((ls[0] + ls[1]) + (ls[2] + ls[3]));
      m_ref = m_use;
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(smem_u32(&bars.p_full[sl][b]));
    }
    // o_done may be two phases behind here, which a parity wait cannot tell apart; o_final has one phase.
    if (ok) ok = wait_w(smem_u32(&bars.o_final[sl]), 0);
    if (ok) {
      tc_fence_after();
      const float inv = 1.f / l_sum;
      __nv_bfloat16* dst = o + ((int64_t)(qt.q_start + row) * n_q_heads + hq) * kD;
#pragma unroll
      for (int c = 0; c < kD / 32; ++c) {
        uint32_t t[32];
        tmem_ld32(t_lane + kColO + sl * 128 + 32 * c, t);
        tc_wait_ld();
        if (row_valid) {
#pragma unroll
          for (int x = 0; x < 32; x += 8) {
            uint4 u;
            u.x = pack_bf16(__uint_as_float(t[x + 0]) * inv, __uint_as_float(t[x + 1]) * inv);
            u.y = pack_bf16(__uint_as_float(t[x + 2]) * inv, __uint_as_float(t[x + 3]) * inv);
            u.z = pack_bf16(__uint_as_float(t[x + 4]) * inv, __uint_as_float(t[x + 5]) * inv);
            u.w = pack_bf16(__uint_as_float(t[x + 6]) * inv, __uint_as_float(t[x + 7]) * inv);
            *reinterpret_cast<uint4*>(dst + 32 * c + x) = u;
          }
        }
      }
      if (lse && row_valid)
        lse[(int64_t)hq * hdr->total_tokens + qt.q_start + row] = (m_ref + log2f(l_sum)) * 0.6931471805599453f;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
  if (tid == 0 && abort_s && start_ok) atomicExch(status, (int32_t)PUREKV_ERR_TIMEOUT);
}

// ---- host side ------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// [T, heads, 128] bf16 -> 3-D map (dim, head, token), box 64 x 1 x rows, 128-byte swizzle, zero fill.
static purekv_status make_map(CUtensorMap* map, const void* base, int64_t n_tokens, int32_t heads, int32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  PK_REQUIRE(fn != nullptr, PUREKV_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  const cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)heads, (cuuint64_t)n_tokens};
  const cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)heads * kD * 2};
  const cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  PK_REQUIRE(r == CUDA_SUCCESS, PUREKV_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  return PUREKV_OK;
}

__device__ int32_t g_default_status;

template <int BK>
static purekv_status launch(const PrefillArgs& a, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                            int32_t* status) {
  const size_t smem = 1024 + 2 * 2 * (size_t)kBQ * 128 + 2 * (size_t)Cfg<BK>::kStages * 2 * BK * 128;
  PK_CUDA(cudaFuncSetAttribute(prefill_tc_kernel<BK>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const int32_t G = a.n_q_heads / a.n_kv_heads;
  dim3 grid((unsigned)((int64_t)a.info->n_qtiles * a.n_kv_heads * ((G + 1) / 2)));
  prefill_tc_kernel<BK><<<grid, kThreads, smem, a.stream>>>(mq, mk, mv, (__nv_bfloat16*)a.o, a.lse,
                                                            (const uint8_t*)a.plan, a.n_q_heads, a.n_kv_heads,
                                                            a.scale * 1.4426950408889634f, status);
  PK_CUDA(cudaGetLastError());
  return PUREKV_OK;
}

}  // namespace tc

purekv_status launch_prefill_tc(const PrefillArgs& a) {
  using namespace tc;
  PK_REQUIRE(a.info->tile_q == kBQ && (a.info->tile_k == 64 || a.info->tile_k == 128) && a.head_dim == kD,
             PUREKV_ERR_UNSUPPORTED, "tensor-core prefill needs tile_q 128, tile_k 64/128, head_dim 128");
  const int64_t T = a.batch->total_tokens;
  CUtensorMap mq, mk, mv;
  purekv_status st;
  if ((st = make_map(&mq, a.q, T, a.n_q_heads, kBQ)) != PUREKV_OK) return st;
  if ((st = make_map(&mk, a.k, T, a.n_kv_heads, a.info->tile_k)) != PUREKV_OK) return st;
  if ((st = make_map(&mv, a.v, T, a.n_kv_heads, a.info->tile_k)) != PUREKV_OK) return st;
  int32_t* status = a.status;
  if (!status) PK_CUDA(cudaGetSymbolAddress((void**)&status, g_default_status));
  return a.info->tile_k == 64 ? launch<64>(a, mq, mk, mv, status) : launch<128>(a, mq, mk, mv, status);
}

}  // namespace purekv
