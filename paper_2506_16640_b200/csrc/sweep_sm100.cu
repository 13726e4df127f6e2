// Score sweep for bf16 problems on sm_100a: S = Q K^T on tcgen05 tensor cores (bf16 in, fp32
// accumulators in TMEM, Q and K tiles staged by TMA without multicast), one pass over the keys of
// every query row, leaving short per-row candidate lists that provably contain the support of
// Eq. 1.
//
// Why one pass is enough.  Write y_j = (alpha-1) s_ij and f(tau) = sum_j [y_j - tau]_+^e - 1, e = 1/(alpha-1).
//  (1) p_max <= 1 gives tau >= y_max - 1 (lower end of the bracket of App. A), and
//  (2) the threshold of a subset of the row's keys never exceeds the threshold of the whole row (adding
//      a logit never lowers tau), while keys at or below the threshold do not change it.
// So while the keys stream by, a thread keeps a lower bound thr on the row's final tau and the list of
// the keys it has seen with y > thr.  When a list grows past kHalfTrigger entries, Newton steps on the
// listed keys, started at thr, raise thr (f is convex and decreasing for e >= 1, so Newton from the left
// of the root never passes it) and the list is filtered.  A row whose list cannot be brought down to
// kHalfKeep entries is flagged and later recomputed by the dense-row path.  In backward mode the
// threshold is the tau of the forward pass and the lists are simply the support.
//
// CTA layout (576 threads, one CTA per SM, persistent; work items of 2 x 128 query rows are handed out
// longest-first through an atomic counter):
//   warp 0        scheduler + TMA producer: the item's two Q tiles, K tiles of 256 keys through a ring
//   warp 1        MMA issuer: per K tile one M=128 x N=256 accumulation per Q tile into its own 256
//                 TMEM columns (2 accumulators = all 512 columns).  N = 256 keeps the operand traffic of
//                 an MMA (A 4 KB + B 8 KB per 128 tensor-core cycles) below the shared-memory bandwidth.
//   warps 2..17   consumers, eight warps per Q tile: TMEM lane = query row; the 256 columns of a row are
//                 split between two threads (columns 0-127 and 128-255 of every K tile), each with its
//                 own running maximum, threshold, list length (registers) and half-list; the two share
//                 their running maxima through shared memory so that both thresholds stay tight.
// A consumer first reduces its 128 columns to 16 group maxima (branch-free), and only when some lane of
// the warp saw a value above its threshold re-reads the groups that hold candidates (four groups per
// round trip to TMEM); it hands the accumulator back as soon as the last values it needs are in registers.  While the consumers of one Q tile scan, the tensor core works on the other.
// Every mbarrier wait is bounded: on expiry the CTA raises ENTMAX_ATTN_FLAG_WAIT_EXPIRED, all roles
// leave their loops, the producer waits for the copies it armed barriers for and the MMA issuer for the tensor-core
// work it issued (each with a bound of its own), TMEM is freed and the CTA returns.
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace entmax {

namespace {

constexpr int BM = 128;          // query rows per Q tile = TMEM lanes
constexpr int BN = 256;          // keys per K tile = N of one MMA = TMEM columns of one accumulator
constexpr int kHalfCols = BN / 2;   // columns of a K tile one consumer thread scans
constexpr int kQTiles = 2;       // Q tiles per item
constexpr int kItemRows = BM * kQTiles;
constexpr int kConsumerWarps = 8 * kQTiles;
constexpr int kThreads = (2 + kConsumerWarps) * 32;
constexpr int kTmemCols = kQTiles * BN;
constexpr int kSchedSlots = 2;
static_assert(kTmemCols == 512 && kHalfCols == 128, "TMEM budget / consumer split");

template <int HD>
struct Cfg {
  static constexpr int kHalves = HD / 64;                 // 64 bf16 = one 128-byte swizzle row
  static constexpr int kQBytes = BM * HD * 2;
  static constexpr int kKBytes = BN * HD * 2;
  static constexpr int kStages = HD == 128 ? 2 : 4;
  static constexpr int kShareBytes = kQTiles * 2 * BM * 8;   // running maxima shared by the two halves of a row
  static constexpr int kBarBytes = 512;
  static constexpr int kSmemBytes = kQTiles * kQBytes + kStages * kKBytes + kShareBytes + 1024 /*align*/ + kBarBytes;
};

struct SweepArgs {
  int B, H, N;
  int causal;
  int mode;             // 0: search the threshold; 1: threshold given (tau_in)
  int expo_class;
  float expo;
  float alpha_m1;       // alpha - 1
  float sm_scale;
  const float* scale;   // [H, N] (scale_sb = 0) or [B, H, N] (scale_sb = H*N)
  long long scale_sb;
  const float* tau_in;  // [B*H*N] (mode 1)
  int32_t* half_cnt;    // [B*H*N][2] list length of each half-row; -1 = hand the row to the dense path
  float* half_thr;      // [B*H*N][2] lower bound on tau each half-row ended with (Eq. 1's units)
  Entry* entries;       // [B*H*N][kListCap]; half h of a row owns slots [h*kHalfCap, (h+1)*kHalfCap)
  float* dump;          // kDump kernels: optional [N, N] raw accumulators of head dump_bh; kAlibi kernels: the
                        // [H] ALiBi slopes m_h (z_ij += m_h (j - i), j <= i).  One member for both keeps the
                        // argument block, and with it the register allocation of the plain kernel, unchanged
  int dump_bh;
  int32_t* status;
  int32_t* work_counter;  // zeroed before the launch
  int items_per_bh;     // ceil(N / kItemRows)
  int n_items;
};
// The kernel's argument block (three tensor maps + this struct) is kept at 512 bytes: one more member made
// the compiler's register allocation of the hot loop spill five times as much (measured: 2.3 -> 2.9 ms).
static_assert(sizeof(SweepArgs) + 3 * sizeof(CUtensorMap) <= 512, "keep the sweep kernel's argument block within 512 bytes");

using namespace sm100;

// Instruction descriptor: fp32 accumulate, A and B bf16, both K-major, M = 128, N = BN
__host__ __device__ constexpr uint32_t make_idesc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}


// --------------------------------------------------------------------------------- work schedule
// Items are handed out in the order k = 0, 1, ...: head pair after head pair (so that the CTAs running at
// the same time stream the same K tiles through L2) and, under the causal mask, the longest rows of a
// head pair first.
__device__ __forceinline__ void decode_item(const SweepArgs& a, int k, int& bh, int& item) {
  bh = k / a.items_per_bh;
  const int w = k - bh * a.items_per_bh;
  item = a.causal ? a.items_per_bh - 1 - w : w;
}
// K tiles Q tile x of an item has to see (0 when the Q tile lies past the end of the sequence)
__device__ __forceinline__ int qtile_tiles(const SweepArgs& a, int item, int x) {
  const int row0 = item * kItemRows + x * BM;
  if (row0 >= a.N) return 0;
  if (!a.causal) return (a.N + BN - 1) / BN;
  int last_row = row0 + BM - 1;
  if (last_row > a.N - 1) last_row = a.N - 1;
  return last_row / BN + 1;
}

// Sampled tiles.  In forward mode an item first scores its query rows against every kSampleStride-th
// key (a second view of K: the key index split into (index / stride, index % stride), phase 0 taken),
// maxima only: the running maxima and thresholds the real stream then starts from are already close to
// their final values, which roughly halves the candidates it pushes (a one-pass stream pushes every new
// running maximum, about ln n of them per row; after a 1/16 sample about ln 16 are left; measured best among 8, 16, 32, 64).
constexpr int kSampleStride = 8;
constexpr int kSampleMinKeys = 4096;   // below this the stream is too short for the sample to pay
__device__ __forceinline__ int sample_tiles(const SweepArgs& a, int item) {
  if (a.mode != 0) return 0;
  int last_row = item * kItemRows + kItemRows - 1;
  if (last_row > a.N - 1) last_row = a.N - 1;
  const int n_vis = a.causal ? last_row + 1 : a.N;
  if (n_vis < kSampleMinKeys) return 0;
  int groups = (n_vis + kSampleStride - 1) / kSampleStride;
  if (groups > a.N / kSampleStride) groups = a.N / kSampleStride;
  return (groups + BN - 1) / BN;
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}

// ALiBi window (kAlibi kernels).  The penalty m_h (i - j) grows with the distance, so keys farther back than a
// bound cannot reach the support (the paper's hard cutoff d_max for entmax + ALiBi): alibi_window_kernel below
// finds, per work item, the first K tile that can still hold a candidate, and all three roles start there.
// In those kernels `dump` points to a blob in the workspace: float slopes [H], then int32 first tiles [n_items].
template <bool kAlibi>
__device__ __forceinline__ int first_tile(const SweepArgs& a, int k) {
  if constexpr (kAlibi) return reinterpret_cast<const int32_t*>(a.dump)[a.H + k];
  return 0;
}

// ------------------------------------------------------------- consumer side: one half-row per thread
struct RowState {
  float thr;       // candidates are accumulators above this (accumulator units)
  float m_run;     // running maximum accumulator (both halves of the row, as far as known)
  int cnt;         // half-list length; -1 = handed to the dense path
};

// Warp-cooperative list shrink for the lanes whose half-list has grown past kHalfTrigger.  Accumulator
// units are turned into Eq. 1's units with y = a * acc.  All 32 lanes must call this together.
// Takes and returns the row state by value: a state whose address escaped would have to be kept in
// local memory across every asm statement of the scan loop.
__device__ __noinline__ RowState shrink_lists(RowState r, Entry* list, float a, float inv_a, unsigned need, int mode,
                                              int expo_class, float expo) {
  const int lane = threadIdx.x & 31;
  constexpr int kSlots = kHalfCap / 32;
  __syncwarp();   // the owner's list stores are ordered before the other lanes' loads
  while (need) {
    const int src = __ffs(need) - 1;
    need &= need - 1;
    Entry* l = reinterpret_cast<Entry*>(__shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(list), src));
    const int c = __shfl_sync(0xffffffffu, r.cnt, src);
    const float th = __shfl_sync(0xffffffffu, r.thr, src);
    const float aa = __shfl_sync(0xffffffffu, a, src);
    const float inv_aa = __shfl_sync(0xffffffffu, inv_a, src);
    float new_thr = INFINITY;
    int kept = -1;
    if (mode == 0) {
      Entry e[kSlots];
#pragma unroll
      for (int s = 0; s < kSlots; ++s) {
        const int idx = lane + 32 * s;
        e[s].y = -INFINITY;
        e[s].j = 0;
        if (idx < c) e[s] = l[idx];
      }
      // A sure case first.  With y_max the largest of the c listed keys, sum_j (y_max - tau)^e >= sum_j [y_j - tau]_+^e
      // = 1 at the list's own threshold tau*, so tau* <= y_max - c^(-1/e): every listed key above that is in the
      // list's support.  If those alone are more than a half-list may keep, the row goes to the dense path without a
      // solve (rows of flat logits, which would otherwise each pay a full Newton solve just to be handed over).
      bool sure_dense = false;
      {
        float ym = -INFINITY;
#pragma unroll
        for (int s = 0; s < kSlots; ++s) ym = fmaxf(ym, e[s].y);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ym = fmaxf(ym, __shfl_xor_sync(0xffffffffu, ym, o));
        const float width = expo_class == kExpo2 ? rsqrtf((float)c) : expo_class == kExpo1 ? 1.0f / (float)c
                                                                                           : powf((float)c, -1.0f / expo);
        const float cut = ym - width * inv_aa;
        int sure = 0;
#pragma unroll
        for (int s = 0; s < kSlots; ++s) sure += __popc(__ballot_sync(0xffffffffu, e[s].y > cut));
        sure_dense = sure > kHalfKeep;
      }
      float tau = th * aa;
      if (sure_dense) {
        // nothing to solve
      } else if (expo >= 1.0f) {
        for (int it = 0; it < 8; ++it) {
          float s0 = 0.f, s1 = 0.f;
#pragma unroll
          for (int s = 0; s < kSlots; ++s) {
            const float y = fmaf(aa, e[s].y, -tau);
            if (y > 0.f) {
              float ye, ye1;
              pow_pair(y, expo_class, expo, ye, ye1);
              s0 += ye;
              s1 += ye1;
            }
          }
          s0 = warp_sum(s0);
          s1 = warp_sum(s1);
          if (!(s0 > 1.0f) || !(s1 > 0.f)) break;
          const float step = threshold_step(s0, s1, expo_class, expo);
          tau += step;
          if (step <= 1e-4f) break;
        }
      } else {
        // e < 1 (alpha > 2): plain bisection between the current bound (mass of the listed keys >= 1 there) and one
        // unit above it (tau <= y_max <= bound + 1); the lower end stays a valid bound whatever the rounding does
        float lo = tau, hi = tau + 1.0f;
        for (int it = 0; it < 14; ++it) {
          const float mid = 0.5f * (lo + hi);
          float s0 = 0.f;
#pragma unroll
          for (int s = 0; s < kSlots; ++s) {
            const float y = fmaf(aa, e[s].y, -mid);
            if (y > 0.f) s0 += powf(y, expo);
          }
          s0 = warp_sum(s0);
          if (s0 > 1.0f) lo = mid; else hi = mid;
        }
        tau = lo;
      }
      // a hair below the Newton iterate: rounding must never push the bound past the true threshold
      new_thr = fmaxf(th, (tau - 4e-6f * fmaxf(1.0f, fabsf(tau))) * inv_aa);
      __syncwarp();
      kept = 0;
      if (!sure_dense) {
#pragma unroll
        for (int s = 0; s < kSlots; ++s) {
          const bool keep = e[s].y > new_thr;
          const unsigned m = __ballot_sync(0xffffffffu, keep);
          if (keep) l[kept + __popc(m & ((1u << lane) - 1u))] = e[s];
          kept += __popc(m);
        }
      }
      if (kept > kHalfKeep || sure_dense) {
        kept = -1;
        new_thr = INFINITY;
      }
    }
    if (lane == src) {
      r.cnt = kept;
      r.thr = new_thr;
    }
  }
  __syncwarp();
  return r;
}

template <int HD, bool kDump, bool kAlibi>
__global__ void __launch_bounds__(kThreads, 1) sweep_kernel(const __grid_constant__ CUtensorMap map_q,
                                                            const __grid_constant__ CUtensorMap map_k,
                                                            const __grid_constant__ CUtensorMap map_ks,
                                                            const SweepArgs a) {
  using C = Cfg<HD>;
  extern __shared__ uint8_t smem_raw[];
  // everything in shared memory is addressed by 32-bit shared-window addresses derived from one base
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_smem = sbase;                                   // [kQTiles][kHalves][BM rows x 128 B]
  const uint32_t k_smem = sbase + kQTiles * C::kQBytes;            // [kStages][kHalves][BN rows x 128 B]
  // running maximum of each half-row, tagged with the work item it belongs to: {item id, float bits}
  const uint32_t m_share = k_smem + C::kStages * C::kKBytes;       // u64 [kQTiles][2][BM]
  const uint32_t bars = m_share + C::kShareBytes;                  // mbarriers, 8 bytes each
  const uint32_t q_full = bars;                            // [kQTiles]
  const uint32_t q_empty = q_full + 8 * kQTiles;           // [kQTiles]
  const uint32_t s_full = q_empty + 8 * kQTiles;           // [kQTiles]
  const uint32_t s_empty = s_full + 8 * kQTiles;           // [kQTiles]
  const uint32_t k_full = s_empty + 8 * kQTiles;           // [kStages]
  const uint32_t k_empty = k_full + 8 * C::kStages;        // [kStages]
  const uint32_t w_full = k_empty + 8 * C::kStages;        // [kSchedSlots]
  const uint32_t w_empty = w_full + 8 * kSchedSlots;       // [kSchedSlots]
  const uint32_t w_item = w_empty + 8 * kSchedSlots;       // int32 [kSchedSlots]
  const uint32_t tmem_slot = w_item + 4 * kSchedSlots;     // uint32
  const uint32_t abort_flag = tmem_slot + 4;               // uint32
  const uint32_t drain_bar = tmem_slot + 8;                // teardown: "every MMA issued so far has finished"
  const uint32_t drain_fail = drain_bar + 8;               // uint32: a teardown wait ran out as well
  static_assert((4 * kQTiles + 2 * C::kStages + 2 * kSchedSlots) * 8 + kSchedSlots * 4 + 8 + 16 <= C::kBarBytes,
                "barrier area");

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int t = 0; t < kQTiles; ++t) {
      mbar_init(q_full + 8 * t, 1);
      mbar_init(q_empty + 8 * t, 1);
      mbar_init(s_full + 8 * t, 1);
      mbar_init(s_empty + 8 * t, 8);                 // one arrival per consumer warp of the Q tile
    }
    for (int t = 0; t < C::kStages; ++t) {
      mbar_init(k_full + 8 * t, 1);
      mbar_init(k_empty + 8 * t, 1);
    }
    for (int t = 0; t < kSchedSlots; ++t) {
      mbar_init(w_full + 8 * t, 1);
      mbar_init(w_empty + 8 * t, 1 + kConsumerWarps);   // MMA issuer + one arrival per consumer warp
    }
    mbar_init(drain_bar, 1);
    sts_u32(abort_flag, 0u);
    sts_u32(drain_fail, 0u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (threadIdx.x < kQTiles * 2 * BM) sts_u64(m_share + 8 * threadIdx.x, ~0ull);   // tag -1: belongs to no work item
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = lds_u32(tmem_slot);

  if (warp == 0) {
    // ------------------------------------------------------------- scheduler + TMA producer
    // (the whole warp runs the control flow, one elected lane issues the copies: see the MMA issuer)
    {
      int stage = 0, slot = 0;
      uint32_t kphase = 0, qphase = 0 /* bit x: phase of Q tile slot x */, wphase = 0;
      bool alive = true;
      auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
      };
      while (alive) {
        alive = wait_all(w_empty + 8 * slot, wphase ^ 1u);
        if (!alive) break;
        int k = 0;
        if (lane == 0) {
          k = atomicAdd(a.work_counter, 1);
          if (k >= a.n_items) k = -1;
          sts_u32(w_item + 4 * slot, (uint32_t)k);
          mbar_arrive(w_full + 8 * slot);
        }
        k = __shfl_sync(0xffffffffu, k, 0);
        if (++slot == kSchedSlots) { slot = 0; wphase ^= 1u; }
        if (k < 0) break;
        int bh, item;
        decode_item(a, k, bh, item);
        const int b = bh / a.H, h = bh - b * a.H;
        int tiles = 0;
        for (int x = 0; x < kQTiles; ++x) {
          const int tx = qtile_tiles(a, item, x);
          tiles = tx > tiles ? tx : tiles;
        }
        // tiles before tf (and sampled tiles before ts0) lie outside the ALiBi window: t counts from there
        const int tf = __shfl_sync(0xffffffffu, first_tile<kAlibi>(a, k), 0);
        const int ts_all = sample_tiles(a, item);
        const int ts0 = kAlibi ? min(tf / kSampleStride, ts_all) : 0;
        const int ts = ts_all - ts0;
        tiles -= tf;
        for (int t = 0; t < ts + tiles && alive; ++t) {
          alive = wait_all(k_empty + 8 * stage, kphase ^ 1u);
          if (!alive) break;
          if (elect_one()) {
            mbar_expect_tx(k_full + 8 * stage, C::kKBytes);
            for (int hf = 0; hf < C::kHalves; ++hf) {
              const uint32_t dst = k_smem + stage * C::kKBytes + hf * (BN * 128);
              if (t < ts) tma_load_5d(dst, &map_ks, k_full + 8 * stage, hf * 64, 0, (ts0 + t) * BN, h, b);
              else tma_load_4d(dst, &map_k, k_full + 8 * stage, hf * 64, (tf + t - ts) * BN, h, b);
            }
          }
          __syncwarp();
          if (++stage == C::kStages) { stage = 0; kphase ^= 1u; }
          if (t == 0) {
            // Q tile slots past the end of the sequence are neither loaded nor used; each slot keeps
            // its own phase bit so that producer and MMA issuer stay in step
            for (int x = 0; x < kQTiles && alive; ++x) {
              if (qtile_tiles(a, item, x) == 0) continue;
              alive = wait_all(q_empty + 8 * x, ((qphase >> x) & 1u) ^ 1u);
              if (!alive) break;
              qphase ^= 1u << x;
              if (elect_one()) {
                mbar_expect_tx(q_full + 8 * x, C::kQBytes);
                for (int hf = 0; hf < C::kHalves; ++hf)
                  tma_load_4d(q_smem + x * C::kQBytes + hf * (BM * 128), &map_q, q_full + 8 * x, hf * 64,
                              item * kItemRows + x * BM, h, b);
              }
              __syncwarp();
            }
          }
        }
      }
      if (!alive && lane == 0) {
        // a wait ran out somewhere in the CTA: every copy this warp armed a barrier for must have landed before
        // shared memory goes away.  Stages before `stage` were armed in this round of the ring, the others in the
        // previous one (a barrier that was never armed reports its "previous" phase as complete at once).
        bool ok = true;
        for (int st = 0; st < C::kStages; ++st) ok &= mbar_drain(k_full + 8 * st, st < stage ? kphase : kphase ^ 1u);
        for (int x = 0; x < kQTiles; ++x) ok &= mbar_drain(q_full + 8 * x, ((qphase >> x) & 1u) ^ 1u);
        if (!ok) sts_u32(drain_fail, 1u);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp runs the control flow (waits are voted on, what is read from shared memory is broadcast), so
    // that descriptors, addresses and counters are warp-uniform; one elected lane issues the tensor-core
    // instructions.
    {
      constexpr uint32_t idesc = make_idesc();
      const uint64_t hi = (uint64_t)kDescHi << 32;
      const uint64_t q_desc = hi | smem_desc_lo(q_smem), k_desc = hi | smem_desc_lo(k_smem);
      int stage = 0, slot = 0;
      uint32_t kphase = 0, qphase = 0, wphase = 0, sphase[kQTiles] = {};
      bool alive = true;
      auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
      };
      while (alive) {
        alive = wait_all(w_full + 8 * slot, wphase);
        if (!alive) break;
        const int k = __shfl_sync(0xffffffffu, (int)lds_u32(w_item + 4 * slot), 0);
        __syncwarp();
        if (lane == 0) mbar_arrive(w_empty + 8 * slot);
        if (++slot == kSchedSlots) { slot = 0; wphase ^= 1u; }
        if (k < 0) break;
        int bh, item;
        decode_item(a, k, bh, item);
        int tx[kQTiles], tiles = 0;
        for (int x = 0; x < kQTiles; ++x) {
          tx[x] = qtile_tiles(a, item, x);
          tiles = tx[x] > tiles ? tx[x] : tiles;
        }
        const int tf = __shfl_sync(0xffffffffu, first_tile<kAlibi>(a, k), 0);
        const int ts_all = sample_tiles(a, item);
        const int ts = ts_all - (kAlibi ? min(tf / kSampleStride, ts_all) : 0);
        tiles -= tf;
        for (int x = 0; x < kQTiles; ++x) tx[x] = tx[x] > 0 ? tx[x] - tf : 0;   // every valid Q tile reaches past tf
        for (int t = 0; t < ts + tiles && alive; ++t) {
          alive = wait_all(k_full + 8 * stage, kphase);
          if (!alive) break;
          const uint64_t b_desc = k_desc + (uint64_t)(stage * (C::kKBytes >> 4));
#pragma unroll
          for (int x = 0; x < kQTiles; ++x) {
            // every valid Q tile takes all sampled tiles, then its own share of the real ones
            if (tx[x] == 0 || t >= ts + tx[x] || !alive) continue;
            if (t == 0) {
              alive = wait_all(q_full + 8 * x, (qphase >> x) & 1u);
              qphase ^= 1u << x;
            }
            if (alive) alive = wait_all(s_empty + 8 * x, sphase[x] ^ 1u);
            if (!alive) continue;
            sphase[x] ^= 1u;
            tc_fence_after();
            const uint64_t a_desc = q_desc + (uint64_t)(x * (C::kQBytes >> 4));
            if (elect_one()) {
#pragma unroll
              for (int kk = 0; kk < HD / 16; ++kk) {
                // k-step kk: 64-column half kk / 4 (its own swizzled block), 32 bytes per step inside the half
                const uint32_t a_off = (kk >> 2) * ((BM * 128) >> 4) + (kk & 3) * 2;
                const uint32_t b_off = (kk >> 2) * ((BN * 128) >> 4) + (kk & 3) * 2;
                umma_bf16_desc(tmem_base + x * BN, a_desc + a_off, b_desc + b_off, idesc, kk > 0 ? 1u : 0u);
              }
              umma_commit(s_full + 8 * x);
              if (t == ts + tx[x] - 1) umma_commit(q_empty + 8 * x);
            }
            __syncwarp();
          }
          if (!alive) break;
          if (elect_one()) umma_commit(k_empty + 8 * stage);
          __syncwarp();
          if (++stage == C::kStages) { stage = 0; kphase ^= 1u; }
        }
      }
      if (!alive && lane == 0) {
        // the tensor core must be done with shared memory and TMEM before they are released
        umma_commit(drain_bar);
        if (!mbar_drain(drain_bar, 0u)) sts_u32(drain_fail, 1u);
      }
    }
  } else {
    // -------------------------------------------------- consumers: one thread per half of a query row
    const int cw = warp - 2;
    const int x = cw >> 3;                         // Q tile of this warp
    const int half = (cw >> 2) & 1;                // which 128 columns of every K tile
    const int quad = warp & 3;                     // TMEM lane quadrant this warp may read
    const int row_local = quad * 32 + lane;
    const uint32_t taddr_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(x * BN + half * kHalfCols);
    const uint32_t my_share = m_share + 8 * ((x * 2 + half) * BM + row_local);
    const uint32_t other_share = m_share + 8 * ((x * 2 + (half ^ 1)) * BM + row_local);
    const uint32_t my_full = s_full + 8 * x, my_empty = s_empty + 8 * x;
    uint32_t fphase = 0, wphase = 0;
    int slot = 0;
    bool alive = true;
    while (alive) {
      alive = __all_sync(0xffffffffu, mbar_wait(w_full + 8 * slot, wphase, abort_flag));
      if (!alive) break;
      const int k = (int)lds_u32(w_item + 4 * slot);
      __syncwarp();
      if (lane == 0) mbar_arrive(w_empty + 8 * slot);
      if (++slot == kSchedSlots) { slot = 0; wphase ^= 1u; }
      if (k < 0) break;
      int bh, item;
      decode_item(a, k, bh, item);
      const int tiles = qtile_tiles(a, item, x);
      if (tiles == 0) continue;
      const int tf = first_tile<kAlibi>(a, k);
      const int h = bh % a.H;
      const int tile_row0 = item * kItemRows + x * BM;
      const int i = tile_row0 + row_local;
      const bool valid = i < a.N;
      const size_t grow = (size_t)bh * a.N + (valid ? i : 0);
      Entry* list = a.entries + grow * kListCap + half * kHalfCap;
      const int lim = a.causal ? i : a.N - 1;      // largest visible key index
      RowState r;
      r.cnt = 0;
      r.m_run = -INFINITY;
      r.thr = INFINITY;
      float ra = 1.f, inv_a = 1.f;
      if (valid) {
        ra = a.alpha_m1 * (a.scale[(size_t)(bh / a.H) * a.scale_sb + (size_t)h * a.N + i] * a.sm_scale);
        if (ra > 0.f && ra < INFINITY) {
          inv_a = 1.0f / ra;
          if (a.mode == 0) {
            r.thr = -INFINITY;
          } else {
            const float t_acc = a.tau_in[grow] * inv_a;
            r.thr = t_acc - 1e-6f * fabsf(t_acc);   // a hair below: the row kernel applies the exact test
          }
        } else {
          r.cnt = -1;   // non-positive or non-finite scale: dense path
        }
      }
      // ALiBi (causal): the logit is sm_scale * (acc + slope * (j - i)); everything below works on that sum
      const float slope = kAlibi ? a.dump[h] / a.sm_scale : 0.f;
      const float fi = (float)i;
      const bool searching = a.mode == 0 && r.cnt == 0 && valid;
      const bool dump_here = kDump && a.dump != nullptr && bh == a.dump_bh && valid;
      // first / last visible key over the rows of this Q tile: halves past the last one are skipped,
      // halves that reach past the first one need the mask
      const int first_lim = a.causal ? tile_row0 : a.N - 1;
      const int last_lim = a.causal ? (tile_row0 + BM - 1 < a.N - 1 ? tile_row0 + BM - 1 : a.N - 1) : a.N - 1;
      // ---- sampled tiles first (forward mode, long rows): maxima only, nothing is pushed -- every sampled
      //      key comes by again in the real stream.  Column c of sampled tile t is key kSampleStride * (t*BN + c).
      const int ts = sample_tiles(a, item);
      const int ts0 = kAlibi ? min(tf / kSampleStride, ts) : 0;
      if (kAlibi && a.status && cw == 0 && lane == 0) {
        // K-tile steps of this item left out by the window / still scored
        const int t_item = max(tiles, qtile_tiles(a, item, kQTiles - 1));
        atomicAdd(a.status + ENTMAX_ATTN_STATUS_SKIPPED_STEPS, tf);
        atomicAdd(a.status + ENTMAX_ATTN_STATUS_SCORED_STEPS, t_item - tf);
      }
      if (ts > ts0) {
        // largest sampled group index that is a key this row may look at
        int glim = lim / kSampleStride;
        if (glim > a.N / kSampleStride - 1) glim = a.N / kSampleStride - 1;
        for (int t = ts0; t < ts && alive; ++t) {
          alive = __all_sync(0xffffffffu, mbar_wait(my_full, fphase, abort_flag));
          if (!alive) break;
          fphase ^= 1u;
          tc_fence_after();
          const int g_base = t * BN + half * kHalfCols;
          float m_s = -INFINITY;
          float va[32];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            tmem_ld32(taddr_row + c * 32, va);
            tmem_ld_wait();
#pragma unroll
            for (int u = 0; u < 32; ++u) {
              if (kAlibi) va[u] = fmaf(slope * (float)kSampleStride, (float)u, va[u]);
              va[u] = (g_base + c * 32 + u <= glim) ? va[u] : -INFINITY;
            }
            float m_c = fmaxf(fmaxf(max8(&va[0]), max8(&va[8])), fmaxf(max8(&va[16]), max8(&va[24])));
            if (kAlibi) m_c += slope * ((float)(kSampleStride * (g_base + c * 32)) - fi);
            m_s = fmaxf(m_s, m_c);
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(my_empty);
          if (searching) {
            const unsigned long long o = lds_u64(other_share);
            const float m_other = (int)(o >> 32) == k ? __uint_as_float((unsigned)o) : -INFINITY;
            r.m_run = max3(r.m_run, m_s, m_other);
            r.thr = fmaxf(r.thr, r.m_run - inv_a);
            sts_u64(my_share, ((unsigned long long)(unsigned)k << 32) | __float_as_uint(r.m_run));
          }
        }
      }
      for (int t = tf; t < tiles && alive; ++t) {
        // the warp leaves together: tcgen05.ld needs all 32 lanes
        alive = __all_sync(0xffffffffu, mbar_wait(my_full, fphase, abort_flag));
        if (!alive) break;
        fphase ^= 1u;
        tc_fence_after();
        const int col_base = t * BN + half * kHalfCols;
        bool released = false;
        if (col_base <= last_lim) {
          const bool masked = col_base + kHalfCols - 1 > first_lim;
          // ---- pass 1: 128 columns -> 16 group maxima (8 columns each); four loads of 32 columns (wider
          //      loads mean fewer TMEM round trips on the path that holds the accumulator)
          float g[16];
          float va[32];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            tmem_ld32(taddr_row + c * 32, va);
            tmem_ld_wait();
            if (kDump) {
              if (dump_here) {
#pragma unroll
                for (int u = 0; u < 32; ++u)
                  if (col_base + c * 32 + u <= lim) a.dump[(size_t)i * a.N + col_base + c * 32 + u] = va[u];
              }
            }
            if (kAlibi) {
              // column part of the bias by an FMA with an immediate; the chunk's constant part joins the maxima
#pragma unroll
              for (int u = 0; u < 32; ++u) va[u] = fmaf(slope, (float)u, va[u]);
            }
            if (masked) {
#pragma unroll
              for (int u = 0; u < 32; ++u) va[u] = (col_base + c * 32 + u <= lim) ? va[u] : -INFINITY;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) g[4 * c + q] = max8(&va[8 * q]);
            if (kAlibi) {
              const float t0 = slope * ((float)(col_base + c * 32) - fi);
#pragma unroll
              for (int q = 0; q < 4; ++q) g[4 * c + q] += t0;
            }
          }
          float m_tile = max3(g[0], g[1], g[2]);
#pragma unroll
          for (int u = 3; u < 15; u += 2) m_tile = max3(m_tile, g[u], g[u + 1]);
          m_tile = fmaxf(m_tile, g[15]);
          if (searching) {
            // the other half's running maximum (if it already belongs to this item) tightens the bound too
            const unsigned long long o = lds_u64(other_share);
            const float m_other = (int)(o >> 32) == k ? __uint_as_float((unsigned)o) : -INFINITY;
            r.m_run = max3(r.m_run, m_tile, m_other);
            if (r.cnt >= 0) r.thr = fmaxf(r.thr, r.m_run - inv_a);
            sts_u64(my_share, ((unsigned long long)(unsigned)k << 32) | __float_as_uint(r.m_run));
          }
          // ---- pass 2 (only when some lane saw a candidate): re-read the groups that hold one
          const bool hit = m_tile > r.thr;
          if (__any_sync(0xffffffffu, hit)) {
            unsigned mine = 0;
#pragma unroll
            for (int u = 0; u < 16; ++u) mine |= (g[u] > r.thr ? 1u : 0u) << u;
            unsigned todo = __reduce_or_sync(0xffffffffu, mine);
            while (todo) {
              // up to four groups per round trip to TMEM (todo is the same in every lane)
              int gu[4];
#pragma unroll
              for (int w = 0; w < 4; ++w) {
                gu[w] = todo ? __ffs(todo) - 1 : -1;
                todo &= todo - 1;
              }
              float v8[4][8];
#pragma unroll
              for (int w = 0; w < 4; ++w)
                if (gu[w] >= 0) tmem_ld8(taddr_row + gu[w] * 8, v8[w]);
              tmem_ld_wait();
              if (todo == 0) {
                // the last batch is in registers: hand the accumulator back before the list stores
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(my_empty);
                released = true;
              }
              if (kAlibi) {
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                  const float tw = slope * ((float)(col_base + gu[w] * 8) - fi);
#pragma unroll
                  for (int e = 0; e < 8; ++e) v8[w][e] = fmaf(slope, (float)e, v8[w][e]) + tw;
                }
              }
              if (masked) {
#pragma unroll
                for (int w = 0; w < 4; ++w)
#pragma unroll
                  for (int e = 0; e < 8; ++e)
                    v8[w][e] = (gu[w] >= 0 && col_base + gu[w] * 8 + e <= lim) ? v8[w][e] : -INFINITY;
              }
#pragma unroll
              for (int w = 0; w < 4; ++w) {
                if (gu[w] >= 0 && ((mine >> gu[w]) & 1u)) {
                  const float thr = r.thr;
                  int cnt = r.cnt;
#pragma unroll
                  for (int e = 0; e < 8; ++e) {
                    if (v8[w][e] > thr) {
                      *reinterpret_cast<uint2*>(&list[cnt]) =
                          make_uint2(__float_as_uint(v8[w][e]), (unsigned)(col_base + gu[w] * 8 + e));
                      ++cnt;
                    }
                  }
                  r.cnt = cnt;
                }
              }
              // at most 32 entries were appended since the last check: the half-list cannot overflow
              const unsigned need = __ballot_sync(0xffffffffu, r.cnt > kHalfTrigger);
              if (need) r = shrink_lists(r, list, ra, inv_a, need, a.mode, a.expo_class, a.expo);
            }
          }
        }
        // the accumulator has been read: hand it back to the MMA issuer (unless pass 2 already did)
        if (!released) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(my_empty);
        }
      }
      if (valid && alive) {
        a.half_cnt[grow * 2 + half] = r.cnt;
        a.half_thr[grow * 2 + half] = r.thr * ra;
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (lds_u32(abort_flag)) {
    if (threadIdx.x == 0 && a.status) atomicOr(a.status + ENTMAX_ATTN_STATUS_FLAGS, ENTMAX_ATTN_FLAG_WAIT_EXPIRED);
    // the producer and the MMA issuer have waited for their copies and MMAs in flight (above); only if one of those
    // waits ran out as well is there nothing left but to give the hardware time
    if (lds_u32(drain_fail)) {
      const uint64_t t0 = global_ns();
      while (global_ns() - t0 < 200000ull) { }
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------- ALiBi window pre-kernels
// Largest key norm of every K tile (BN keys) of every head: kmax[bh * k_tiles + t].
template <int HD>
__global__ void __launch_bounds__(BN) key_norm_kernel(const __nv_bfloat16* __restrict__ k, int H, int N, long long sb,
                                                      long long sh, long long sn, int k_tiles, float* __restrict__ kmax) {
  __shared__ float red[BN / 32];
  const int bh = blockIdx.x / k_tiles, t = blockIdx.x - bh * k_tiles;
  const int b = bh / H, h = bh - b * H;
  const int j = t * BN + threadIdx.x;
  float n2 = 0.f;
  if (j < N) {
    const __nv_bfloat16* row = k + (size_t)b * sb + (size_t)h * sh + (size_t)j * sn;
#pragma unroll
    for (int c = 0; c < HD / 8; ++c) {
      const uint4 raw = *reinterpret_cast<const uint4*>(row + 8 * c);
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[u]));
        n2 = fmaf(f.x, f.x, fmaf(f.y, f.y, n2));
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) n2 = fmaxf(n2, __shfl_xor_sync(0xffffffffu, n2, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = n2;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = red[0];
    for (int w = 1; w < BN / 32; ++w) m = fmaxf(m, red[w]);
    kmax[blockIdx.x] = sqrtf(m);
  }
}

// First K tile of every work item that can hold a candidate.  For row i a lower bound on its threshold is known
// before any score: its own key (distance 0, no penalty) gives tau_i >= y_ii - 1 (App. A bracket), i.e. in
// accumulator units thr_i >= <q_i,k_i> - 1/a_i; in backward mode thr_i is the given tau_i.  A key j of tile t scores at
// most |q_i| max_t|k| - (m_h / sm_scale) (i - j_last(t)) (Cauchy-Schwarz; the slope in accumulator units), so the tile
// is outside row i's support when that is <= thr_i: the paper's hard cutoff d_max for entmax with ALiBi, with the
// logit range bounded by norms.  The item starts at the first tile some row of it still needs.
// blob: float slopes [H] (copied here), then int32 first tiles [n_items].
template <int HD>
__global__ void __launch_bounds__(kItemRows) alibi_window_kernel(const __nv_bfloat16* __restrict__ q,
                                                                 const __nv_bfloat16* __restrict__ k, SweepArgs a,
                                                                 long long sb, long long sh, long long sn,
                                                                 const float* __restrict__ slopes,
                                                                 const float* __restrict__ kmax, int k_tiles,
                                                                 float* __restrict__ blob) {
  __shared__ int red[kItemRows / 32];
  int bh, item;
  decode_item(a, blockIdx.x, bh, item);
  const int b = bh / a.H, h = bh - b * a.H;
  const int i = item * kItemRows + threadIdx.x;
  const float slope = slopes[h] / a.sm_scale;
  int need = item;   // never past the tile that holds the item's first row (and its own key)
  if (i < a.N && slope > 0.f) {
    const size_t base = (size_t)b * sb + (size_t)h * sh + (size_t)i * sn;
    float qq = 0.f, qk = 0.f;
#pragma unroll
    for (int c = 0; c < HD / 8; ++c) {
      const uint4 rq = *reinterpret_cast<const uint4*>(q + base + 8 * c);
      const uint4 rk = *reinterpret_cast<const uint4*>(k + base + 8 * c);
      const uint32_t wq[4] = {rq.x, rq.y, rq.z, rq.w}, wk[4] = {rk.x, rk.y, rk.z, rk.w};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float2 fq = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wq[u]));
        const float2 fk = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wk[u]));
        qq = fmaf(fq.x, fq.x, fmaf(fq.y, fq.y, qq));
        qk = fmaf(fq.x, fk.x, fmaf(fq.y, fk.y, qk));
      }
    }
    const size_t grow = (size_t)bh * a.N + i;
    const float ra = a.alpha_m1 * (a.scale[(size_t)b * a.scale_sb + (size_t)h * a.N + i] * a.sm_scale);
    float thr = INFINITY;          // no usable bound: the row needs every tile
    if (ra > 0.f && ra < INFINITY) {
      thr = a.mode == 0 ? qk - 1.0f / ra : a.tau_in[grow] / ra;
      thr -= 1e-5f * fabsf(thr) + 1e-6f;     // rounding of the dot product and of the bound
    }
    const float qn = sqrtf(qq) * 1.0002f;    // rounding of the norms
    need = 0;
    if (thr < INFINITY) {
      for (; need < item; ++need) {
        const int j_last = need * BN + BN - 1;
        if (j_last >= i) break;
        if (qn * kmax[(size_t)bh * k_tiles + need] - slope * (float)(i - j_last) > thr) break;
      }
    }
  } else if (i < a.N) {
    need = 0;                      // no positional term on this head
  }
  for (int o = 16; o > 0; o >>= 1) need = min(need, __shfl_xor_sync(0xffffffffu, need, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = need;
  __syncthreads();
  if (threadIdx.x == 0) {
    int m = red[0];
    for (int w = 1; w < kItemRows / 32; ++w) m = min(m, red[w]);
    reinterpret_cast<int32_t*>(blob)[a.H + blockIdx.x] = m;
    blob[h] = slopes[h];
  }
}

// cuTensorMapEncodeTiled through the runtime's driver entry point lookup (no link against libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

cudaError_t get_encode_fn(EncodeTiledFn* fn) {
  static EncodeTiledFn cached = nullptr;
  if (!cached) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t err = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres);
    if (err != cudaSuccess) return err;
    if (qres != cudaDriverEntryPointSuccess || !p) return cudaErrorNotSupported;
    cached = reinterpret_cast<EncodeTiledFn>(p);
  }
  *fn = cached;
  return cudaSuccess;
}

// [B,H,N,D] bf16 tensor as a 4-D map (D, N, H, B); box = 64 columns (one 128-byte swizzle row) x rows
cudaError_t make_map(CUtensorMap* map, const void* base, const Problem& p, int box_rows) {
  EncodeTiledFn fn;
  cudaError_t err = get_encode_fn(&fn);
  if (err != cudaSuccess) return err;
  cuuint64_t dims[4] = {(cuuint64_t)p.D, (cuuint64_t)p.N, (cuuint64_t)p.H, (cuuint64_t)p.B};
  cuuint64_t strides[3] = {(cuuint64_t)p.sn * 2, (cuuint64_t)p.sh * 2, (cuuint64_t)p.sb * 2};
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// K as a 5-D map (D, key % stride, key / stride, H, B): a box of BN rows along "key / stride" at phase 0
// is every kSampleStride-th key.  Keys past stride * (N / stride) are not part of the view.
cudaError_t make_sample_map(CUtensorMap* map, const void* base, const Problem& p) {
  EncodeTiledFn fn;
  cudaError_t err = get_encode_fn(&fn);
  if (err != cudaSuccess) return err;
  const cuuint64_t groups = (cuuint64_t)(p.N / kSampleStride);
  cuuint64_t dims[5] = {(cuuint64_t)p.D, (cuuint64_t)kSampleStride, groups > 0 ? groups : 1, (cuuint64_t)p.H,
                        (cuuint64_t)p.B};
  cuuint64_t strides[4] = {(cuuint64_t)p.sn * 2, (cuuint64_t)p.sn * 2 * kSampleStride, (cuuint64_t)p.sh * 2,
                           (cuuint64_t)p.sb * 2};
  cuuint32_t box[5] = {64, 1, (cuuint32_t)BN, 1, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int HD, bool kDump, bool kAlibi>
cudaError_t launch_impl(const Problem& p, const void* q, const void* k, SweepArgs& args, cudaStream_t stream) {
  CUtensorMap map_q, map_k, map_ks;
  cudaError_t err = make_map(&map_q, q, p, BM);
  if (err != cudaSuccess) return err;
  err = make_map(&map_k, k, p, BN);
  if (err != cudaSuccess) return err;
  if (p.N >= kSampleMinKeys) {
    err = make_sample_map(&map_ks, k, p);
    if (err != cudaSuccess) return err;
  } else {
    map_ks = map_k;   // never used: sample_tiles() is 0 for short sequences
  }
  err = cudaFuncSetAttribute(sweep_kernel<HD, kDump, kAlibi>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Cfg<HD>::kSmemBytes);
  if (err != cudaSuccess) return err;
  int dev = 0, sms = 0;
  err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;
  err = cudaMemsetAsync(args.work_counter, 0, sizeof(int32_t), stream);
  if (err != cudaSuccess) return err;
  const int grid = args.n_items < sms ? args.n_items : sms;
  sweep_kernel<HD, kDump, kAlibi><<<grid, kThreads, Cfg<HD>::kSmemBytes, stream>>>(map_q, map_k, map_ks, args);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_sweep(const Problem& p, const void* q, const void* k, const float* scale, const float* tau_in,
                         int mode, int32_t* half_cnt, float* half_thr, Entry* entries, int32_t* work_counter,
                         float* dump, int dump_bh, float* alibi_blob, float* alibi_kmax, int32_t* status,
                         cudaStream_t stream) {
  SweepArgs args;
  args.B = p.B; args.H = p.H; args.N = p.N;
  args.causal = p.causal;
  args.mode = mode;
  args.expo_class = p.expo_class;
  args.expo = p.expo;
  args.alpha_m1 = p.alpha - 1.0f;
  args.sm_scale = p.sm_scale;
  args.scale = scale;
  args.scale_sb = p.scale_sb;
  args.tau_in = tau_in;
  args.half_cnt = half_cnt;
  args.half_thr = half_thr;
  args.entries = entries;
  args.dump = p.alibi ? alibi_blob : dump;
  args.dump_bh = dump_bh;
  args.status = status;
  args.work_counter = work_counter;
  args.items_per_bh = (p.N + kItemRows - 1) / kItemRows;
  args.n_items = args.items_per_bh * p.B * p.H;
  if (p.alibi && !dump) {
    // the window: key norms per K tile, then the first tile of every item (and the slopes) into the blob
    const int k_tiles = (p.N + BN - 1) / BN;
    const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q);
    const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(k);
    if (p.D == 64) {
      key_norm_kernel<64><<<p.B * p.H * k_tiles, BN, 0, stream>>>(kb, p.H, p.N, p.sb, p.sh, p.sn, k_tiles, alibi_kmax);
      alibi_window_kernel<64><<<args.n_items, kItemRows, 0, stream>>>(qb, kb, args, p.sb, p.sh, p.sn, p.alibi, alibi_kmax,
                                                                      k_tiles, alibi_blob);
    } else {
      key_norm_kernel<128><<<p.B * p.H * k_tiles, BN, 0, stream>>>(kb, p.H, p.N, p.sb, p.sh, p.sn, k_tiles, alibi_kmax);
      alibi_window_kernel<128><<<args.n_items, kItemRows, 0, stream>>>(qb, kb, args, p.sb, p.sh, p.sn, p.alibi, alibi_kmax,
                                                                       k_tiles, alibi_blob);
    }
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
  }
  if (dump) return p.D == 64 ? launch_impl<64, true, false>(p, q, k, args, stream)
                             : launch_impl<128, true, false>(p, q, k, args, stream);
  if (p.alibi) return p.D == 64 ? launch_impl<64, false, true>(p, q, k, args, stream)
                                : launch_impl<128, false, true>(p, q, k, args, stream);
  return p.D == 64 ? launch_impl<64, false, false>(p, q, k, args, stream)
                   : launch_impl<128, false, false>(p, q, k, args, stream);
}

}  // namespace entmax
