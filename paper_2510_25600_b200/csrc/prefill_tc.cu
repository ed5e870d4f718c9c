// Tensor-core ST-SpAttn prefill (Sec. 3.2) for bf16, head_dim 128, on sm_100a.
//
// Persistent kernel: one CTA per SM walks the list of work units the plan assigned to it.  A unit is a
// 128-row query tile of a PAIR of query heads that share a KV head ("slots") and a chunk of that tile's
// list of kept key tiles, so every K/V tile staged in shared memory feeds two heads and key blocks the
// mask removes are never read.  With an odd number of heads per KV head the group's last head is worked on by both
// slots for two consecutive query tiles over the union of their lists (a twin unit), each slot with its own tile
// classes and bit masks.  Roles:
//   warp 8      producer: per unit Q of both slots, then per key tile the tile's class word and, for
//               general tiles, its bit mask (bulk copy) into a small ring, and K and V (TMA, 128-byte
//               swizzle, two 64-column panels each) into a ring of stages.  It runs ahead across units.
//   warp 9      owns the 512 TMEM columns; one lane issues tcgen05.mma, alternating slots:
//               S = Q K^T (K-major A and B from shared memory) and
//               O += P V (A = bf16 P from TMEM, B = V as MN-major shared-memory operand),
//               so the tensor pipe works on one slot while the other slot's rows are in softmax.
//   warps 0-7   one thread per query row of a slot (registers raised with setmaxnreg at the expense of
//               warps 8-11): the row of S from TMEM into registers, the
//               tile's predicate (none / causal / bit mask), online softmax in the log2 domain against a
//               reference that moves only when exp2 would overflow (then O is rescaled), a share of the
//               exponentials on the FMA pipe, bf16 P written over S; at the end of a unit either the normalised output
//               (whole list in one unit) or an unnormalised fp32 partial result plus (max, sum) per row
//               into the workspace.  The chunk of a split list that finishes last (a counter in the plan)
//               combines the partial results in chunk order, so the result does not depend on timing.
// Every wait on an mbarrier is bounded in time; on expiry the CTA raises a shared abort flag,
// sets the device status word, drains, frees TMEM and exits.
#include <type_traits>

#include "prefill.cuh"
#include "tc_util.cuh"

namespace purekv {
namespace tc {

constexpr int kBQ = 128;
constexpr int kThreads = 384;  // warps 0-3 softmax of slot 0, warps 4-7 of slot 1, warp 8 producer, warp 9 MMA, 10-11 idle
constexpr int kWarpProducer = 8, kWarpMma = 9;
// Per-thread registers after the warpgroups trade them.  setmaxnreg only moves registers inside the CTA's launch
// allocation (kThreads x the count ptxas gives the kernel, 168 at 384 threads); asking for more would block forever,
// so the launch code checks the budget against the compiled register count.
constexpr int kRegsSoftmax = 208, kRegsOther = 88;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColO = 256;
constexpr int kUnitRing = 4;  // units in flight between the producer's publication and the other roles' copies

template <int BK>
struct Cfg {
  static constexpr int kStages = 2;                 // K/V ring depth (64 KB per stage)
  static constexpr int kSBuf = 128 / BK;            // S buffers per slot: kSBuf * BK = 128 TMEM columns
  static constexpr int kMeta = 2 * kStages;         // ring of per-tile class words and bit masks
  static constexpr uint32_t kMaskBytes = kBQ * BK / 8;
};

template <int BK>
struct __align__(8) Barriers {
  static constexpr int ST = Cfg<BK>::kStages, SB = Cfg<BK>::kSBuf, MR = Cfg<BK>::kMeta;
  uint64_t q_full, q_empty;
  uint64_t k_full[ST], k_empty[ST], v_full[ST], v_empty[ST];
  uint64_t m_full[MR];     // producer -> softmax: class word (and bit mask) of a tile are in place
  uint64_t s_full[2][SB];  // MMA -> softmax: S of (slot, buffer) is complete
  uint64_t p_full[2][SB];  // softmax -> MMA: P written (and O rescaled) by the slot's four row warps
  uint64_t o_done[2];      // one completion per P.V product of the slot
  uint64_t o_final[2];     // one completion per unit, after the slot's last P.V product
  uint64_t rows_sync[2];   // the 128 row threads of a slot meet here around the merge-counter update
  uint64_t u_full[kUnitRing];   // the producer published a unit (or the end mark) in unit_s[]
  uint64_t u_empty[kUnitRing];  // the MMA thread and the eight softmax warps have copied it
  uint64_t drain;
};

// TMEM columns: S(slot, buf) at slot*128 + buf*BK (P aliases its first BK/2 columns), O(slot) at 256 + slot*128.
template <int BK>
__global__ void __launch_bounds__(kThreads, 1) prefill_tc_kernel(
    const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_k64,
    const __grid_constant__ CUtensorMap tm_v64, __nv_bfloat16* __restrict__ o, float* __restrict__ lse,
    uint8_t* __restrict__ plan, float* __restrict__ ws, int32_t n_q_heads, int32_t n_kv_heads, float scale_log2,
    int32_t* __restrict__ status, uint64_t wait_ns, int64_t plan_bytes, int64_t ws_floats) {
  constexpr int ST = Cfg<BK>::kStages, SB = Cfg<BK>::kSBuf, MR = Cfg<BK>::kMeta;
  constexpr uint32_t kPanelQ = kBQ * 128;  // bytes of one 64-column panel of a Q tile
  constexpr uint32_t kTileQ = 2 * kPanelQ;
  constexpr uint32_t kPanelKV = BK * 128;  // bytes of one 64-column panel of a K or V tile
  constexpr uint32_t kTileKV = 2 * kPanelKV;
  constexpr uint32_t kMaskBytes = Cfg<BK>::kMaskBytes;
  extern __shared__ uint8_t smem_raw[];
  __shared__ Barriers<BK> bars;
  __shared__ int2 meta_s[MR][2];  // per slot: the entry word, and the byte offset in shared memory of the slot's bit mask
  __shared__ Unit unit_s[kUnitRing];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  __shared__ int abort_code_s;  // what the status word becomes if the CTA gives up: an expired wait unless set otherwise
  __shared__ int merge_s[2];

  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = smem0;                 // [2 slots][2 panels][128 rows x 128 B]
  const uint32_t sK = sQ + 2 * kTileQ;       // [ST][2 panels][BK rows x 128 B]
  const uint32_t sV = sK + ST * kTileKV;
  const uint32_t sM = sV + ST * kTileKV;     // [MR][2 slots][128 rows x BK/8 B]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // Programmatic dependent launch: the next kernel in the stream may start its CTAs as ours retire and set up its
  // barriers and TMEM meanwhile; nothing the previous kernel may have written is read before griddep_wait below.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  volatile int* abort_flag = &abort_s;

  if (tid == 0) {
    mbar_init(smem_u32(&bars.q_full), 1);
    mbar_init(smem_u32(&bars.q_empty), 1);
    for (int s = 0; s < ST; ++s) {
      mbar_init(smem_u32(&bars.k_full[s]), 1);
      mbar_init(smem_u32(&bars.k_empty[s]), 1);
      mbar_init(smem_u32(&bars.v_full[s]), 1);
      mbar_init(smem_u32(&bars.v_empty[s]), 1);
    }
    for (int s = 0; s < MR; ++s) mbar_init(smem_u32(&bars.m_full[s]), 1);
    for (int sl = 0; sl < 2; ++sl) {
      for (int b = 0; b < SB; ++b) {
        mbar_init(smem_u32(&bars.s_full[sl][b]), 1);
        mbar_init(smem_u32(&bars.p_full[sl][b]), 4);
      }
      mbar_init(smem_u32(&bars.o_done[sl]), 1);
      mbar_init(smem_u32(&bars.o_final[sl]), 1);
      mbar_init(smem_u32(&bars.rows_sync[sl]), 128);
    }
    for (int s = 0; s < kUnitRing; ++s) {
      mbar_init(smem_u32(&bars.u_full[s]), 1);
      mbar_init(smem_u32(&bars.u_empty[s]), 9);
    }
    mbar_init(smem_u32(&bars.drain), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == kWarpMma) {
    tmem_alloc(smem_u32(&tmem_base_s), kTmemCols);
    tmem_relinquish();
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the stream's earlier work is complete and visible from here on
  if (tid == 0) {
    abort_s = *reinterpret_cast<volatile int32_t*>(status) != 0;  // an earlier CTA or launch already failed
    abort_code_s = (int)PUREKV_ERR_TIMEOUT;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  const PlanHeader* hdr = reinterpret_cast<const PlanHeader*>(plan);
  // The plan is checked before anything is read through it: the header's own fields here (by every thread, on the
  // same values, so the decision is uniform), each unit and each list entry by the producer before it publishes or
  // uses them.  A plan that fails is not used: the status word becomes PUREKV_ERR_BAD_PLAN and the CTA leaves.
  bool plan_ok = plan_bytes >= (int64_t)sizeof(PlanHeader);
  if (plan_ok) {
    const int64_t G_ = n_kv_heads > 0 ? n_q_heads / n_kv_heads : 0;
    auto section = [&](int64_t off, int64_t count, int64_t elem) {
      return off >= (int64_t)sizeof(PlanHeader) && (off & 15) == 0 && count >= 0 && count <= plan_bytes / elem &&
             off <= plan_bytes - count * elem;
    };
    plan_ok = hdr->magic == kPlanMagic && hdr->tile_q == kBQ && hdr->tile_k == BK && hdr->words_per_row == BK / 32 &&
              hdr->n_q_heads == n_q_heads && hdr->n_kv_heads == n_kv_heads && G_ >= 1 &&
              hdr->n_ctas == (int32_t)gridDim.x && hdr->n_units >= 1 && hdr->n_counters >= 0 &&
              section(hdr->off_entries, hdr->n_entries, 8) && section(hdr->off_masks, hdr->n_mask_words, 4) &&
              section(hdr->off_units, hdr->n_units, (int64_t)sizeof(Unit)) &&
              section(hdr->off_counters, (int64_t)hdr->n_counters + 2, 4) && hdr->part_slots >= 0 &&
              hdr->part_slots <= ws_floats / kPartFloats && hdr->total_tokens >= 0;
  }
  if (!plan_ok) {
    if (tid == 0 && abort_s == 0) atomicExch(status, (int32_t)PUREKV_ERR_BAD_PLAN);
    hdr = nullptr;
  }
  const int2* entries = reinterpret_cast<const int2*>(plan + (plan_ok ? hdr->off_entries : 0));
  const uint32_t* masks = reinterpret_cast<const uint32_t*>(plan + (plan_ok ? hdr->off_masks : 0));
  const Unit* units = reinterpret_cast<const Unit*>(plan + (plan_ok ? hdr->off_units : 0));
  int32_t* counters = reinterpret_cast<int32_t*>(plan + (plan_ok ? hdr->off_counters : 0));
  const int32_t G = n_q_heads / n_kv_heads, ppg = (G + 1) >> 1;
  // Units are handed out at run time: CTA c starts with unit c of the list (sorted by decreasing cost) and draws
  // every further one from a counter behind the merge counters, so the CTAs finish within one small unit of one
  // another whatever the units really cost.  The producer draws and publishes; the other roles follow unit_s[].
  const int32_t n_units = plan_ok ? hdr->n_units : 0;
  int32_t* sched = counters + (plan_ok ? hdr->n_counters : 0);  // [0] units drawn beyond the first round, [1] CTAs that drew their last
  const int64_t n_entries = plan_ok ? hdr->n_entries : 0, n_mask_words = plan_ok ? hdr->n_mask_words : 0;
  const int64_t total_tokens = plan_ok ? hdr->total_tokens : 0;
  const int32_t n_counters = plan_ok ? hdr->n_counters : 0;
  const int64_t part_slots = plan_ok ? hdr->part_slots : 0;
  const bool withhold_first_k = plan_ok && (hdr->test_flags & 1u) != 0u;
  const bool start_ok = abort_s == 0 && plan_ok;
  // the two softmax warpgroups take registers from the warpgroup of the producer and MMA warps

  if (warp >= 8) {
    setmaxnreg_dec<kRegsOther>();
  if (start_ok && warp == kWarpProducer) {
    // ---------------- producer (whole warp; lane 0 issues) ----------------
    uint32_t it = 0;  // key tiles issued so far by this CTA, over all units
    int32_t issued_k = 0, issued_v = 0;
    bool ok = true;
    // unit idx of the list, or the end mark (ent_count 0) past its end
    // Also checks the unit: a unit whose fields point outside the plan's sections, the batch or the workspace is not
    // published; the CTA gives up with PUREKV_ERR_BAD_PLAN instead.
    auto fetch = [&](int32_t idx) -> Unit {
      Unit uu = {};
      if (idx < n_units) {
        uu = units[idx];
        const int32_t n_pairs = n_kv_heads * ppg;
        const bool split = uu.n_chunks > 1, twin = uu.q_rows1 != 0;
        const bool good = uu.ent_count >= 1 && uu.ent_begin >= 0 &&
                          (int64_t)uu.ent_begin + (int64_t)uu.ent_count * (twin ? 2 : 1) <= n_entries &&
                          uu.q_rows >= 1 && uu.q_rows <= kBQ && uu.req_start >= 0 && uu.q_start >= uu.req_start &&
                          (int64_t)uu.q_start + uu.q_rows <= total_tokens && uu.pair >= 0 && uu.pair < n_pairs &&
                          uu.n_chunks >= 1 && uu.chunk >= 0 && uu.chunk < uu.n_chunks &&
                          (!twin || (uu.q_rows1 >= 1 && uu.q_rows1 <= kBQ && uu.q_start1 >= uu.req_start &&
                                     (int64_t)uu.q_start1 + uu.q_rows1 <= total_tokens && (G & 1) != 0 &&
                                     uu.pair % ppg == ppg - 1 &&
                                     (!split || (uu.part_base1 >= 0 && ((int64_t)uu.part_base1 + uu.n_chunks) * n_q_heads <= part_slots &&
                                                 uu.counter_base1 >= 0 && (int64_t)uu.counter_base1 + n_q_heads <= n_counters)))) &&
                          (!split || (uu.part_base >= 0 && ((int64_t)uu.part_base + uu.n_chunks) * n_q_heads <= part_slots &&
                                      uu.counter_base >= 0 && (int64_t)uu.counter_base + n_q_heads <= n_counters));
        if (!good) {
          abort_code_s = (int)PUREKV_ERR_BAD_PLAN;
          *abort_flag = 1;
          uu = Unit{};
        }
      }
      return uu;
    };
    // lane 0: put a fetched unit into the ring as the CTA's unit number uo
    auto publish = [&](const Unit& uu, uint32_t uo) -> bool {
      if (*abort_flag) return false;
      const uint32_t us = uo % kUnitRing;
      if (uo >= (uint32_t)kUnitRing && !mbar_wait(smem_u32(&bars.u_empty[us]), ((uo / kUnitRing) - 1u) & 1u, abort_flag, wait_ns))
        return false;
      unit_s[us] = uu;
      mbar_arrive(smem_u32(&bars.u_full[us]));
      if (uu.ent_count == 0) {
        // This CTA has drawn for the last time.  The CTA that does so last of all rewinds both counters for the
        // plan's next launch (nobody reads them any more in this one).
        __threadfence();
        if (atomicAdd(sched + 1, 1) == (int32_t)gridDim.x - 1) {
          sched[0] = 0;
          sched[1] = 0;
        }
      }
      return true;
    };
    if (lane == 0) ok = publish(fetch((int32_t)blockIdx.x), 0u);
    for (uint32_t uo = 0;; ++uo) {
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      __syncwarp();
      const Unit u = unit_s[uo % kUnitRing];
      if (u.ent_count == 0) break;
      // The next unit is drawn as late as the latencies allow: when this unit's last tile goes out (the other roles
      // still have about two tiles of it to work through, which covers the counter's and the list's round trips).
      // Drawn at the start of a unit it would be reserved for as long as that unit runs, and the CTAs with the
      // longest units would keep work from those that finish early.
      int32_t idx_next = 0;
      const int32_t nt = u.ent_count;
      const int32_t g = u.pair / ppg, hq0 = g * G + 2 * (u.pair % ppg);
      const bool twin = u.q_rows1 != 0;  // both slots on head hq0, slot 1 on the query tile at q_start1
      const int32_t n_slots = (twin || 2 * (u.pair % ppg) + 1 < G) ? 2 : 1;
      if (lane == 0) {
        if (uo > 0) ok = mbar_wait(smem_u32(&bars.q_empty), (uo - 1u) & 1u, abort_flag, wait_ns);
        if (ok) {
          mbar_expect_tx(smem_u32(&bars.q_full), n_slots * kTileQ);
          for (int sl = 0; sl < n_slots; ++sl) {
            const int32_t hq = twin ? hq0 : hq0 + sl, qs = (twin && sl) ? u.q_start1 : u.q_start;
            tma_load_3d(sQ + sl * kTileQ, &tm_q, smem_u32(&bars.q_full), 0, hq, qs);
            tma_load_3d(sQ + sl * kTileQ + kPanelQ, &tm_q, smem_u32(&bars.q_full), 64, hq, qs);
          }
        }
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      for (int32_t n0 = 0; ok && n0 < nt; n0 += 32) {
        int2 e_l = make_int2(0, -1), f_l = e_l;  // the tile's entry as slot 0 and as slot 1 see it
        if (n0 + lane < nt) {
          if (twin) {
            e_l = __ldg(entries + u.ent_begin + 2 * (n0 + lane));
            f_l = __ldg(entries + u.ent_begin + 2 * (n0 + lane) + 1);
          } else {
            e_l = f_l = __ldg(entries + u.ent_begin + n0 + lane);
          }
        }
        const int32_t n1 = min(nt, n0 + 32);
        for (int32_t n = n0; ok && n < n1; ++n) {
          int2 e, f;
          e.x = __shfl_sync(0xffffffffu, e_l.x, n - n0);
          e.y = __shfl_sync(0xffffffffu, e_l.y, n - n0);
          f.x = __shfl_sync(0xffffffffu, f_l.x, n - n0);
          f.y = __shfl_sync(0xffffffffu, f_l.y, n - n0);
          if (lane == 0) {
            if (n == nt - 1) idx_next = atomicAdd(sched, 1) + (int32_t)gridDim.x;  // used after the loop
            const uint32_t s = it % ST, par = ((it / ST) - 1u) & 1u, ms = it % MR;
            const int32_t tok = u.req_start + (e.x >> 4) * BK;
            const uint32_t hm = (uint32_t)((e.x | f.x) >> 2) & 3u;  // which 64-key halves of the tile are present
            // the entry is checked before its mask offset or key-tile index is used for a copy: a class the slot
            // knows (none only in a twin unit, and then without halves), a bit mask inside the table
            auto entry_ok = [&](const int2& x) {
              const int32_t c = x.x & 3;
              const uint32_t h = (uint32_t)(x.x >> 2) & 3u;
              if (x.x < 0 || (c == kTileNone ? (!twin || h != 0u) : h == 0u)) return false;
              return c != kTileGeneral ||
                     (x.y >= 0 && (int64_t)x.y + (int64_t)(kMaskBytes / 4) <= n_mask_words && (x.y & 3) == 0);
            };
            if (!entry_ok(e) || !entry_ok(f) || (e.x >> 4) != (f.x >> 4) || hm == 0u || (int64_t)tok >= total_tokens) {
              abort_code_s = (int)PUREKV_ERR_BAD_PLAN;
              *abort_flag = 1;
              ok = false;
            }
            if (ok && it >= (uint32_t)ST) ok = mbar_wait(smem_u32(&bars.k_empty[s]), par, abort_flag, wait_ns);
            if (ok) {
              // a slot's bit mask goes to its own buffer; outside twin units both slots read the first one
              const uint32_t m_off = (sM - smem_u32(smem_raw)) + ms * 2u * kMaskBytes;
              const bool mask0 = (e.x & 3) == kTileGeneral, mask1 = twin && (f.x & 3) == kTileGeneral;
              meta_s[ms][0] = make_int2(e.x, (int32_t)m_off);
              meta_s[ms][1] = make_int2(f.x, (int32_t)(m_off + (twin ? kMaskBytes : 0u)));
              if (mask0 || mask1) {
                mbar_expect_tx(smem_u32(&bars.m_full[ms]), (mask0 && mask1) ? 2u * kMaskBytes : kMaskBytes);
                if (mask0) bulk_load(sM + ms * 2u * kMaskBytes, masks + e.y, kMaskBytes, smem_u32(&bars.m_full[ms]));
                if (mask1)
                  bulk_load(sM + ms * 2u * kMaskBytes + kMaskBytes, masks + f.y, kMaskBytes, smem_u32(&bars.m_full[ms]));
              } else {
                mbar_arrive(smem_u32(&bars.m_full[ms]));
              }
              if (withhold_first_k && it == 0u) {
                // test plans only: this tile's K is never asked for, so whoever waits for it runs into the limit
              } else if (hm == 3u) {
                mbar_expect_tx(smem_u32(&bars.k_full[s]), kTileKV);
                tma_load_3d(sK + s * kTileKV, &tm_k, smem_u32(&bars.k_full[s]), 0, g, tok);
                tma_load_3d(sK + s * kTileKV + kPanelKV, &tm_k, smem_u32(&bars.k_full[s]), 64, g, tok);
              } else {  // one half: 64 rows into their place inside each panel
                const uint32_t hh = hm >> 1, off = hh * (kPanelKV / 2);
                mbar_expect_tx(smem_u32(&bars.k_full[s]), kTileKV / 2);
                tma_load_3d(sK + s * kTileKV + off, &tm_k64, smem_u32(&bars.k_full[s]), 0, g, tok + 64 * (int32_t)hh);
                tma_load_3d(sK + s * kTileKV + kPanelKV + off, &tm_k64, smem_u32(&bars.k_full[s]), 64, g,
                            tok + 64 * (int32_t)hh);
              }
              if (!(withhold_first_k && it == 0u)) issued_k = (int32_t)it + 1;
              if (it >= (uint32_t)ST) ok = mbar_wait(smem_u32(&bars.v_empty[s]), par, abort_flag, wait_ns);
            }
            if (ok) {
              if (hm == 3u) {
                mbar_expect_tx(smem_u32(&bars.v_full[s]), kTileKV);
                tma_load_3d(sV + s * kTileKV, &tm_v, smem_u32(&bars.v_full[s]), 0, g, tok);
                tma_load_3d(sV + s * kTileKV + kPanelKV, &tm_v, smem_u32(&bars.v_full[s]), 64, g, tok);
              } else {
                const uint32_t hh = hm >> 1, off = hh * (kPanelKV / 2);
                mbar_expect_tx(smem_u32(&bars.v_full[s]), kTileKV / 2);
                tma_load_3d(sV + s * kTileKV + off, &tm_v64, smem_u32(&bars.v_full[s]), 0, g, tok + 64 * (int32_t)hh);
                tma_load_3d(sV + s * kTileKV + kPanelKV + off, &tm_v64, smem_u32(&bars.v_full[s]), 64, g,
                            tok + 64 * (int32_t)hh);
              }
              issued_v = (int32_t)it + 1;
            }
          }
          ++it;
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
      }
      if (lane == 0 && ok) ok = publish(fetch(idx_next), uo + 1u);
    }
    if (lane == 0 && *abort_flag) {
      // drain: every issued copy must have landed before shared memory is released
      const uint64_t t0 = global_ns();
      for (int32_t n = max(0, issued_k - ST); n < issued_k; ++n)
        while (!mbar_try_wait(smem_u32(&bars.k_full[n % ST]), (n / ST) & 1) && global_ns() - t0 < wait_ns) {}
      for (int32_t n = max(0, issued_v - ST); n < issued_v; ++n)
        while (!mbar_try_wait(smem_u32(&bars.v_full[n % ST]), (n / ST) & 1) && global_ns() - t0 < wait_ns) {}
      for (int32_t n = max(0, issued_k - MR); n < issued_k; ++n)
        while (!mbar_try_wait(smem_u32(&bars.m_full[n % MR]), (n / MR) & 1) && global_ns() - t0 < wait_ns) {}
      __nanosleep(20000);  // a Q tile possibly still in flight (its barrier's phase is not known here)
    }
  } else if (start_ok && warp == kWarpMma) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(BK, false);
      constexpr uint32_t idesc_qk_half = instr_desc(BK / 2, false);
      constexpr uint32_t idesc_pv = instr_desc(kD, true);
      uint32_t it_base = 0;            // key tiles of earlier units
      uint32_t tq[2] = {0, 0};         // S products issued per slot, over all units
      uint32_t tp[2] = {0, 0};         // P.V products issued per slot, over all units
      int32_t nt = 0, n_slots = 0;
      int32_t pend_v = -1;             // V stage whose release is due behind the next S product
      // Descriptor words.  High word: stride between 8-row groups 1024 B, descriptor version 1, 128-byte swizzle.
      // Low word: start address / 16 and the leading-dimension offset / 16 (used by the MN-major V operand only).
      constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
      const uint32_t q_lo0 = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
      const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
      const uint32_t v_lo0 = ((sV & 0x3FFFFu) >> 4) | ((kPanelKV >> 4) << 16);
      // S(slot, n) = Q_slot K_n^T; the last slot to read K_n releases its stage
      auto issue_qk = [&](auto sl_c, int32_t n) -> bool {
        constexpr int sl = decltype(sl_c)::value;  // compile-time slot: the per-slot counters stay in registers
        const uint32_t it = it_base + (uint32_t)n;
        const uint32_t s = it % ST, b = tq[sl] % SB;
        // the stage was already awaited for slot 0 of the same tile
        if (sl == 0 && !mbar_wait(smem_u32(&bars.k_full[s]), (it / ST) & 1u, abort_flag, wait_ns)) return false;
        tc_fence_after();
        const uint32_t hm = (uint32_t)((meta_s[it % MR][0].x | meta_s[it % MR][1].x) >> 2) & 3u;  // written before the stage's barrier was armed
        const uint32_t q_lo = q_lo0 + (uint32_t)sl * (kTileQ >> 4);
        if (hm == 3u) {
          const uint32_t d_addr = tmem + sl * 128 + b * BK, k_lo = k_lo0 + s * (kTileKV >> 4);
#pragma unroll
          for (int ks = 0; ks < kD / 16; ++ks)
            mma_ss_lh(d_addr, q_lo + (ks >> 2) * (kPanelQ >> 4) + (ks & 3) * 2, kDescHi,
                      k_lo + (ks >> 2) * (kPanelKV >> 4) + (ks & 3) * 2, kDescHi, idesc_qk, ks > 0 ? 1u : 0u);
        } else {  // one 64-key half: N = 64, into that half's columns of S
          const uint32_t hh = hm >> 1;
          const uint32_t d_addr = tmem + sl * 128 + b * BK + hh * 64;
          const uint32_t k_lo = k_lo0 + s * (kTileKV >> 4) + hh * (kPanelKV >> 5);
#pragma unroll
          for (int ks = 0; ks < kD / 16; ++ks)
            mma_ss_lh(d_addr, q_lo + (ks >> 2) * (kPanelQ >> 4) + (ks & 3) * 2, kDescHi,
                      k_lo + (ks >> 2) * (kPanelKV >> 4) + (ks & 3) * 2, kDescHi, idesc_qk_half, ks > 0 ? 1u : 0u);
        }
        // A commit costs the issuing thread about as long as a product and the slot's rows are waiting for S, so S
        // is announced first; the releases behind it (and the V release a preceding P.V left pending) cover the
        // same products and only reach the producer a little later.
        tc_commit(smem_u32(&bars.s_full[sl][b]));
        if (pend_v >= 0) {
          tc_commit(smem_u32(&bars.v_empty[pend_v]));
          pend_v = -1;
        }
        if (sl == n_slots - 1) {
          tc_commit(smem_u32(&bars.k_empty[s]));
          if (n == nt - 1) tc_commit(smem_u32(&bars.q_empty));  // the unit's last read of Q
        }
        ++tq[sl];
        return true;
      };
      // O(slot) += P(slot, n) V_n; the last slot to read V_n releases its stage
      auto issue_pv = [&](auto sl_c, int32_t n) -> bool {
        constexpr int sl = decltype(sl_c)::value;
        const uint32_t it = it_base + (uint32_t)n;
        const uint32_t s = it % ST, b = tp[sl] % SB;
        if (sl == 0 && !mbar_wait(smem_u32(&bars.v_full[s]), (it / ST) & 1u, abort_flag, wait_ns)) return false;
        // P of the unit's first tile also implies that the previous unit's output has left TMEM
        if (!mbar_wait(smem_u32(&bars.p_full[sl][b]), (tp[sl] / SB) & 1u, abort_flag, wait_ns)) return false;
        tc_fence_after();
        const uint32_t p_addr = tmem + sl * 128 + b * BK, o_addr = tmem + kColO + sl * 128;
        // B = V tile, MN-major: per K step 16 key rows (2 groups of 8, 1024 B apart) x 128 dims (2 panels)
        const uint32_t v_lo = v_lo0 + s * (kTileKV >> 4);
        const uint32_t hm = (uint32_t)((meta_s[it % MR][0].x | meta_s[it % MR][1].x) >> 2) & 3u;
        const uint32_t acc0 = n > 0 ? 1u : 0u;  // the unit's first product overwrites O
        if (hm == 3u) {
#pragma unroll
          for (int ks = 0; ks < BK / 16; ++ks)
            mma_ts_lh(o_addr, p_addr + ks * 8, v_lo + ks * (2048 >> 4), kDescHi, idesc_pv, ks > 0 ? 1u : acc0);
        } else {  // the K steps of the present half only
          const uint32_t k0 = (hm >> 1) * (BK / 32);
#pragma unroll
          for (int ks = 0; ks < BK / 32; ++ks)
            mma_ts_lh(o_addr, p_addr + (k0 + ks) * 8, v_lo + (k0 + ks) * (2048 >> 4), kDescHi, idesc_pv, ks > 0 ? 1u : acc0);
        }
        if (SB > 1) tc_commit(smem_u32(&bars.o_done[sl]));
        if (n == nt - 1) tc_commit(smem_u32(&bars.o_final[sl]));
        if (sl == n_slots - 1) {
          // the V stage is released behind the S product that follows, if one does (see issue_qk)
          if (n + SB < nt) pend_v = (int32_t)s;
          else tc_commit(smem_u32(&bars.v_empty[s]));
        }
        ++tp[sl];
        return true;
      };
      bool ok = true;
      for (uint32_t uo = 0; ok; ++uo) {
        const uint32_t us = uo % kUnitRing;
        if (!mbar_wait(smem_u32(&bars.u_full[us]), (uo / kUnitRing) & 1u, abort_flag, wait_ns)) { ok = false; break; }
        const Unit u = unit_s[us];
        mbar_arrive(smem_u32(&bars.u_empty[us]));
        if (u.ent_count == 0) break;
        nt = u.ent_count;
        n_slots = (u.q_rows1 != 0 || 2 * (u.pair % ppg) + 1 < G) ? 2 : 1;
        ok = mbar_wait(smem_u32(&bars.q_full), uo & 1u, abort_flag, wait_ns);
        constexpr std::integral_constant<int, 0> s0{};
        constexpr std::integral_constant<int, 1> s1{};
        for (int32_t n = 0; ok && n < SB && n < nt; ++n) {
          ok = issue_qk(s0, n);
          if (ok && n_slots == 2) ok = issue_qk(s1, n);
        }
        for (int32_t n = 0; ok && n < nt; ++n) {
          ok = issue_pv(s0, n);
          if (ok && n + SB < nt) ok = issue_qk(s0, n + SB);  // in order behind P.V of tile n, which frees S(slot, n % SB)
          if (ok && n_slots == 2) {
            ok = issue_pv(s1, n);
            if (ok && n + SB < nt) ok = issue_qk(s1, n + SB);
          }
        }
        it_base += (uint32_t)nt;
      }
      if (!ok) {
        // leaving early: let every issued MMA finish before TMEM is released
        tc_commit(smem_u32(&bars.drain));
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(smem_u32(&bars.drain), 0) && global_ns() - t0 < wait_ns) {}
      }
    }
  }
  } else {
    setmaxnreg_inc<kRegsSoftmax>();
  if (start_ok) {
    // ---------------- softmax / epilogue: one thread per query row of one slot ----------------
    const int sl = warp >> 2;
    const int quad = warp & 3;  // TMEM lane quadrant this warp may access
    const int row = quad * 32 + lane;
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16);
    // waits are made warp-uniform: the TMEM loads/stores below need the whole warp
    auto wait_w = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, wait_ns) ? 1 : 0) != 0;
    };
    uint32_t it_base = 0;     // key tiles of earlier units (both slots)
    uint32_t t = 0;           // tiles this slot has processed, over all units
    uint32_t slot_units = 0;  // units this slot took part in
    uint32_t row_syncs = 0;   // completed phases of rows_sync[sl]
    bool ok = true;
    // bounded meeting of the slot's 128 row threads (a plain barrier could not be left on a failure)
    auto sync_rows = [&]() -> bool {
      mbar_arrive(smem_u32(&bars.rows_sync[sl]));
      const bool r = wait_w(smem_u32(&bars.rows_sync[sl]), row_syncs & 1u);
      ++row_syncs;
      return r;
    };
    for (uint32_t uo = 0; ok; ++uo) {
      const uint32_t us = uo % kUnitRing;
      if (!wait_w(smem_u32(&bars.u_full[us]), (uo / kUnitRing) & 1u)) { ok = false; break; }
      // read in place (the fields wanted after the tile loop are not held in registers meanwhile); the ring slot is
      // given back at the end of the unit
      const Unit& u = unit_s[us];
      auto release_unit = [&]() {
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars.u_empty[us]));
      };
      const int32_t nt = u.ent_count;
      if (nt == 0) break;
      const int32_t pr = u.pair % ppg, g = u.pair / ppg;
      const bool twin = u.q_rows1 != 0;
      const int32_t n_slots = (twin || 2 * pr + 1 < G) ? 2 : 1;
      if (sl >= n_slots) {
        // A single-head unit: this slot sits it out.  It takes no part in the tile ring meanwhile: a parity wait only
        // tells a barrier's current phase from the one before, and a slot with nothing to deliver is held back by
        // nobody, so it could fall (or run) a whole ring away from the producer.  The unit ring is a full handshake
        // instead, and the next unit is published only after every tile of this one has been issued, which puts the
        // slot's next tile within the ring's reach again.
        it_base += (uint32_t)nt;
        release_unit();
        continue;
      }
      const int32_t hq = g * G + 2 * pr + (twin ? 0 : sl);
      const bool second = twin && sl == 1;  // this slot works on the unit's second query tile
      const bool row_valid = row < (second ? u.q_rows1 : u.q_rows);
      const int32_t i_rel = (second ? u.q_start1 : u.q_start) - u.req_start + row;
      float m_ref = 0.f, l_sum = 0.f;
      for (int32_t n = 0; n < nt; ++n) {
        const uint32_t it = it_base + (uint32_t)n, ms = it % MR, b = t % SB;
        if (!wait_w(smem_u32(&bars.m_full[ms]), (it / MR) & 1u)) { ok = false; break; }
        const int2 e = meta_s[ms][sl];
        const int32_t cls = e.x & 3, j0 = (e.x >> 4) * BK;
        // hm: the 64-key halves that were loaded and multiplied (chunk c belongs to half c / 2); hm_own: those in which
        // this slot's query tile keeps anything (they differ in twin units only)
        const uint32_t hm_own = (uint32_t)(e.x >> 2) & 3u;
        const uint32_t hm = (uint32_t)((e.x | meta_s[ms][sl ^ 1].x) >> 2) & 3u;
        uint32_t keep[BK / 32];
        if (cls == kTileGeneral) {  // this row's bits of the tile's mask
          const uint32_t* mrow = reinterpret_cast<const uint32_t*>(smem_raw + e.y) + row * (BK / 32);
          static_assert(BK == 128, "a mask row is four 32-bit words");
          const uint4 w4 = *reinterpret_cast<const uint4*>(mrow);
          keep[0] = w4.x; keep[1] = w4.y; keep[2] = w4.z; keep[3] = w4.w;
        } else if (cls == kTileDiag) {
          const int32_t n_ok = min(BK, max(0, i_rel - j0 + 1));  // causal: columns 0 .. n_ok-1
#pragma unroll
          for (int c = 0; c < BK / 32; ++c) {
            const int32_t k_in = min(32, max(0, n_ok - 32 * c));
            keep[c] = k_in >= 32 ? 0xFFFFFFFFu : ((1u << k_in) - 1u);
          }
        } else {
#pragma unroll
          for (int c = 0; c < BK / 32; ++c) keep[c] = 0xFFFFFFFFu;
        }
        if (hm_own != 3u) {  // columns of a half the slot keeps nothing of (or that is absent altogether): masked
#pragma unroll
          for (int c = 0; c < BK / 32; ++c)
            if (!((hm_own >> (c >> 1)) & 1u)) keep[c] = 0u;
        }
        if (!wait_w(smem_u32(&bars.s_full[sl][b]), (t / SB) & 1u)) { ok = false; break; }
        tc_fence_after();
        const uint32_t s_addr = t_lane + sl * 128 + b * BK;
        // Fast path: exponentials against the row's standing reference m_ref, no maximum taken.  Softmax does not depend
        // on the reference, and fp32 / bf16 carry 8 exponent bits, so the reference (0 at the start of a unit) only has
        // to keep exp2 in range: it moves when a tile overflows, or when everything kept so far has underflowed; those
        // tiles take the exact path below.
        uint32_t pk[BK / 2];
        float l_tile = 0.f;
        bool exact = false;
        {
          float2 ls2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
          const float2 sc2 = make_float2(scale_log2, scale_log2), mm2 = make_float2(-m_ref, -m_ref);
          // exponentials of one 64-key half whose S values are in r
          auto half_exp = [&](uint32_t (&r)[64], auto hh_c) {
            constexpr int hh = decltype(hh_c)::value;
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
              constexpr int c0 = 2 * hh;
              const int c = c0 + cc;
              if (cls != kTileFull && __any_sync(0xffffffffu, keep[c] != 0xFFFFFFFFu)) {  // warp-uniform
#pragma unroll
                for (int x = 0; x < 32; ++x)
                  if (!((keep[c] >> x) & 1u)) r[32 * cc + x] = 0xFF800000u;  // -inf: exp2 gives 0
              }
#pragma unroll
              for (int x = 0; x < 32; x += 2) {
                const float2 a = __ffma2_rn(make_float2(__uint_as_float(r[32 * cc + x]), __uint_as_float(r[32 * cc + x + 1])), sc2, mm2);
                // kPolyOf8 of every 8 column pairs take the polynomial on the FMA pipe, the rest the MUFU unit
                const float2 pp = ((x >> 1) & 7) < kPolyOf8 ? exp2_poly2(a) : make_float2(ex2(a.x), ex2(a.y));
                ls2[(x >> 1) & 1] = __fadd2_rn(ls2[(x >> 1) & 1], pp);
                pk[16 * c + (x >> 1)] = pack_bf16(pp.x, pp.y);
              }
            }
          };
          if (hm == 3u) {  // both halves: all loads in flight before the one wait
            uint32_t r0[64], r1[64];
            tmem_ld32_at<0>(s_addr, r0);
            tmem_ld32_at<32>(s_addr + 32, r0);
            tmem_ld32_at<0>(s_addr + 64, r1);
            tmem_ld32_at<32>(s_addr + 96, r1);
            tc_wait_ld();
            half_exp(r0, std::integral_constant<int, 0>{});
            half_exp(r1, std::integral_constant<int, 1>{});
          } else {
            uint32_t r[64];
            tmem_ld32_at<0>(s_addr + (hm >> 1) * 64, r);
            tmem_ld32_at<32>(s_addr + (hm >> 1) * 64 + 32, r);
            tc_wait_ld();
            if (hm == 1u) half_exp(r, std::integral_constant<int, 0>{});
            else half_exp(r, std::integral_constant<int, 1>{});
          }
          l_tile = (ls2[0].x + ls2[0].y) + (ls2[1].x + ls2[1].y);
          bool has_kept = cls == kTileFull;  // (a full tile has both halves)
#pragma unroll
          for (int c = 0; c < BK / 32; ++c) has_kept |= keep[c] != 0u;
          // overflow (inf or NaN), or kept keys and still nothing representable: redo against the true maximum
          exact = __any_sync(0xffffffffu, !(l_tile <= 1.0e30f) || (has_kept && l_sum + l_tile < 1.0e-30f));
        }
        if (exact) {
          // Exact path (rare): re-reference the row; O and the running sum are rescaled.  S is still intact in TMEM
          // (P has not been stored yet).
          float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < BK / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(s_addr + 32 * c, r);
            tc_wait_ld();
#pragma unroll
            for (int x = 0; x < 32; ++x)
              if ((keep[c] >> x) & 1u) mx[x & 3] = fmaxf(mx[x & 3], __uint_as_float(r[x]));
          }
          const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale_log2;  // scale > 0
          // the new reference: the larger of this tile's maximum and the log-sum of what has been accumulated
          const float m_eff = l_sum > 0.f ? m_ref + log2f(l_sum) : -INFINITY;
          const float m_max = fmaxf(m_eff, m_tile);
          const float m_new = m_max == -INFINITY ? m_ref : m_max;  // nothing kept yet and nothing accumulated: stay
          const float alpha = l_sum > 0.f ? ex2(m_ref - m_new) : 1.f;  // with l_sum == 0 every earlier P was 0, so O is 0
          const float m_sub = m_new;
          if (n > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
            // O must be quiescent: with one S buffer, S of tile n was issued behind P.V of tile n-1, so it is;
            // with two, S of tile n only implies P.V of tile n-2 (o_done is then in phase t-1 or t).
            if (SB > 1 && !wait_w(smem_u32(&bars.o_done[sl]), (t - 1u) & 1u)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < kD / 32; ++c) {
              uint32_t tt[32];
              tmem_ld32(t_lane + kColO + sl * 128 + 32 * c, tt);
              tc_wait_ld();
#pragma unroll
              for (int x = 0; x < 32; ++x) tt[x] = __float_as_uint(__uint_as_float(tt[x]) * alpha);
              tmem_st32(t_lane + kColO + sl * 128 + 32 * c, tt);
            }
          }
          float ls[2] = {0.f, 0.f};
#pragma unroll
          for (int c = 0; c < BK / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(s_addr + 32 * c, r);
            tc_wait_ld();
#pragma unroll
            for (int x = 0; x < 32; x += 2) {
              const float p0 = ((keep[c] >> x) & 1u) ? ex2(fmaf(__uint_as_float(r[x]), scale_log2, -m_sub)) : 0.f;
              const float p1 = ((keep[c] >> (x + 1)) & 1u) ? ex2(fmaf(__uint_as_float(r[x + 1]), scale_log2, -m_sub)) : 0.f;
              ls[(x >> 1) & 1] += p0 + p1;
              pk[16 * c + (x >> 1)] = pack_bf16(p0, p1);
            }
          }
          l_tile = ls[0] + ls[1];
          l_sum *= alpha;
          m_ref = m_new;
        }
        l_sum += l_tile;
        // bf16 P over the first BK/2 columns of S, which this thread has consumed
#pragma unroll
        for (int c = 0; c < BK / 32; ++c)
          if ((hm >> (c >> 1)) & 1u) tmem_st16(s_addr + 16 * c, reinterpret_cast<const uint32_t(&)[16]>(pk[16 * c]));
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars.p_full[sl][b]));  // one arrival per warp: 4 per slot
        ++t;
      }
      if (!ok) break;
      it_base += (uint32_t)nt;
      // o_done may be two phases behind here, which a parity wait cannot tell apart; o_final moves once per unit.
      if (!wait_w(smem_u32(&bars.o_final[sl]), slot_units & 1u)) { ok = false; break; }
      ++slot_units;
      tc_fence_after();
      const int32_t q_first = (u.q_rows1 != 0 && sl == 1) ? u.q_start1 : u.q_start;  // the slot's query tile
      if (u.n_chunks == 1) {
        const float inv = 1.f / l_sum;
        __nv_bfloat16* dst = o + ((int64_t)(q_first + row) * n_q_heads + hq) * kD;
#pragma unroll
        for (int c = 0; c < kD / 32; ++c) {
          uint32_t tt[32];
          tmem_ld32(t_lane + kColO + sl * 128 + 32 * c, tt);
          tc_wait_ld();
          if (row_valid) {
#pragma unroll
            for (int x = 0; x < 32; x += 16) {
              uint32_t w[8];
#pragma unroll
              for (int y = 0; y < 8; ++y)
                w[y] = pack_bf16(__uint_as_float(tt[x + 2 * y]) * inv, __uint_as_float(tt[x + 2 * y + 1]) * inv);
              st_global_v8(dst + 32 * c + x, w);
            }
          }
        }
        if (lse && row_valid)
          lse[(int64_t)hq * total_tokens + q_first + row] = (m_ref + log2f(l_sum)) * 0.6931471805599453f;
      } else {
        // one chunk of a split list: leave the unnormalised result for whoever arrives last
        const bool second_tile = u.q_rows1 != 0 && sl == 1;  // a twin unit's second tile has slots and counters of its own
        const int32_t part_base = second_tile ? u.part_base1 : u.part_base;
        float* part = ws + ((int64_t)(part_base + u.chunk) * n_q_heads + hq) * kPartFloats;
#pragma unroll
        for (int c = 0; c < kD / 32; ++c) {
          uint32_t tt[32];
          tmem_ld32(t_lane + kColO + sl * 128 + 32 * c, tt);
          tc_wait_ld();
#pragma unroll
          for (int x = 0; x < 32; x += 4)
            *reinterpret_cast<uint4*>(part + ((c * 8 + (x >> 2)) * 128 + row) * 4) =
                make_uint4(tt[x], tt[x + 1], tt[x + 2], tt[x + 3]);
        }
        part[128 * 128 + row] = m_ref;
        part[128 * 128 + 128 + row] = l_sum;
        // The 128 rows meet (ordering their stores before row 0 inside the CTA), then row 0 alone publishes with one
        // release / acquire update of the merge counter at GPU scope: release is cumulative over what the meeting
        // ordered before it, so no thread needs a fence of its own.
        if (!sync_rows()) { ok = false; break; }
        if (row == 0) {
          int32_t* cnt = counters + (second_tile ? u.counter_base1 : u.counter_base) + hq;
          const int last = atom_add_acq_rel(cnt, 1) == u.n_chunks - 1;
          if (last) *cnt = 0;  // every chunk has arrived: ready for the next launch (nobody touches it before then)
          merge_s[sl] = last;
        }
        if (!sync_rows()) { ok = false; break; }
        if (merge_s[sl]) {
          const float* p0 = ws + ((int64_t)part_base * n_q_heads + hq) * kPartFloats;
          const int64_t cstride = (int64_t)n_q_heads * kPartFloats;
          float m_all = -INFINITY;
          for (int32_t c = 0; c < u.n_chunks; ++c) {
            const float lc = __ldcg(p0 + c * cstride + 128 * 128 + 128 + row);
            const float mc = __ldcg(p0 + c * cstride + 128 * 128 + row);
            if (lc > 0.f) m_all = fmaxf(m_all, mc);
          }
          float l_all = 0.f;
          for (int32_t c = 0; c < u.n_chunks; ++c) {
            const float lc = __ldcg(p0 + c * cstride + 128 * 128 + 128 + row);
            const float mc = __ldcg(p0 + c * cstride + 128 * 128 + row);
            if (lc > 0.f) l_all += lc * ex2(mc - m_all);
          }
          const float inv = 1.f / l_all;
          __nv_bfloat16* dst = o + ((int64_t)(q_first + row) * n_q_heads + hq) * kD;
#pragma unroll 1
          for (int cc = 0; cc < kD / 32; ++cc) {
            float acc[32];
#pragma unroll
            for (int x = 0; x < 32; ++x) acc[x] = 0.f;
            for (int32_t c = 0; c < u.n_chunks; ++c) {
              const float lc = __ldcg(p0 + c * cstride + 128 * 128 + 128 + row);
              const float mc = __ldcg(p0 + c * cstride + 128 * 128 + row);
              const float wgt = lc > 0.f ? ex2(mc - m_all) : 0.f;
              const float* pc = p0 + c * cstride;
#pragma unroll
              for (int x = 0; x < 32; x += 4) {
                const float4 v4 = __ldcg(reinterpret_cast<const float4*>(pc + ((cc * 8 + (x >> 2)) * 128 + row) * 4));
                acc[x] = fmaf(wgt, v4.x, acc[x]);
                acc[x + 1] = fmaf(wgt, v4.y, acc[x + 1]);
                acc[x + 2] = fmaf(wgt, v4.z, acc[x + 2]);
                acc[x + 3] = fmaf(wgt, v4.w, acc[x + 3]);
              }
            }
            if (row_valid) {
#pragma unroll
              for (int x = 0; x < 32; x += 8) {
                uint4 w;
                w.x = pack_bf16(acc[x + 0] * inv, acc[x + 1] * inv);
                w.y = pack_bf16(acc[x + 2] * inv, acc[x + 3] * inv);
                w.z = pack_bf16(acc[x + 4] * inv, acc[x + 5] * inv);
                w.w = pack_bf16(acc[x + 6] * inv, acc[x + 7] * inv);
                *reinterpret_cast<uint4*>(dst + 32 * cc + x) = w;
              }
            }
          }
          if (lse && row_valid)
            lse[(int64_t)hq * total_tokens + q_first + row] = (m_all + log2f(l_all)) * 0.6931471805599453f;
        }
      }
      release_unit();
    }
  }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kWarpMma) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
  if (tid == 0 && abort_s && start_ok) atomicCAS(status, 0, (int32_t)abort_code_s);  // the first code raised stays
}

static purekv_status launch(const PrefillArgs& a, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                            const CUtensorMap& mk64, const CUtensorMap& mv64, int32_t* status) {
  constexpr int BK = 128;
  const size_t smem = 1024 + 2 * 2 * (size_t)kBQ * 128 + 2 * (size_t)Cfg<BK>::kStages * 2 * BK * 128 +
                      2 * (size_t)Cfg<BK>::kMeta * Cfg<BK>::kMaskBytes;
  static std::atomic<int> launch_regs{0};  // the compiled register count: the same on every device, read once
  int regs = launch_regs.load(std::memory_order_relaxed);
  if (regs == 0) {
    cudaFuncAttributes fa;
    PK_CUDA(cudaFuncGetAttributes(&fa, prefill_tc_kernel<BK>));
    regs = fa.numRegs;
    launch_regs.store(regs, std::memory_order_relaxed);
  }
  PK_REQUIRE(256 * kRegsSoftmax + 128 * kRegsOther <= kThreads * regs, PUREKV_ERR_UNSUPPORTED,
             "prefill kernel was compiled with %d registers per thread, too few for its register hand-over", regs);
  {
    static std::atomic<uint64_t> smem_allowed{0};
    const purekv_status st_smem = allow_max_dynamic_smem(prefill_tc_kernel<BK>, smem_allowed);
    if (st_smem != PUREKV_OK) return st_smem;
  }
  dim3 grid((unsigned)a.info->n_ctas);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = a.stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see griddepcontrol in the kernel
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  PK_CUDA(cudaLaunchKernelEx(&cfg, prefill_tc_kernel<BK>, mq, mk, mv, mk64, mv64, (__nv_bfloat16*)a.o, a.lse,
                             (uint8_t*)a.plan, (float*)a.ws, a.n_q_heads, a.n_kv_heads,
                             a.scale * 1.4426950408889634f, status, wait_limit_ns(), (int64_t)a.info->bytes_used,
                             (int64_t)(a.ws_bytes / sizeof(float))));
  PK_CUDA(cudaGetLastError());
  return PUREKV_OK;
}

}  // namespace tc

purekv_status launch_prefill_tc(const PrefillArgs& a) {
  using namespace tc;
  PK_REQUIRE(a.info->tile_q == kBQ && (a.info->tile_k == 64 || a.info->tile_k == 128) && a.head_dim == kD,
             PUREKV_ERR_UNSUPPORTED, "tensor-core prefill needs tile_q 128, tile_k 64/128, head_dim 128");
  PK_REQUIRE(a.info->n_ctas >= 1 && a.info->n_units >= 1, PUREKV_ERR_INVALID_ARG, "plan holds no schedule");
  PK_REQUIRE((uintptr_t)a.o % 32 == 0, PUREKV_ERR_INVALID_ARG, "O must be 32-byte aligned for the tensor-core kernel");
  const int64_t T = a.batch->total_tokens;
  CUtensorMap mq, mk, mv, mk64, mv64;
  purekv_status st;
  if ((st = make_map(&mq, a.q, T, a.n_q_heads, kBQ)) != PUREKV_OK) return st;
  if ((st = make_map(&mk, a.k, T, a.n_kv_heads, 128)) != PUREKV_OK) return st;
  if ((st = make_map(&mv, a.v, T, a.n_kv_heads, 128)) != PUREKV_OK) return st;
  if ((st = make_map(&mk64, a.k, T, a.n_kv_heads, 64)) != PUREKV_OK) return st;
  if ((st = make_map(&mv64, a.v, T, a.n_kv_heads, 64)) != PUREKV_OK) return st;
  int32_t* status = a.status;
  if (!status) {
    const purekv_status st_w = default_status_word(&status);
    if (st_w != PUREKV_OK) return st_w;
  }
  return launch(a, mq, mk, mv, mk64, mv64, status);
}

}  // namespace purekv
