// Dense-tile forward for bf16 problems on sm_100a: the rows whose support does not fit the sparse
// lists of the score sweep are recomputed tile by tile on the tensor cores, the way the method reads
// when nothing is known about the sparsity:
//   threshold   tau_i by Newton from the left on f(tau) = sum_j [y_ij - tau]_+^e - 1 (Eq. 1 with the
//               sum-to-one condition), every iteration one sweep S = Q K^T over the visible K tiles
//               (tcgen05, fp32 accumulators in TMEM), started at the lower end of the bracket of
//               App. A, tau >= y_max - 1, which a first sweep finds;
//   output      one more sweep: P = [y - tau]_+^e, rounded to bf16 and written to shared memory as the
//               A operand of a second tcgen05 contraction O += P V (V tile as the N-major B operand),
//               O accumulated in TMEM over all K tiles.
// A work item is one Q tile of 128 rows that holds at least one such row (a list written by the row
// kernel); only the rows flagged there are written back.
//
// CTA: warp 0 TMA producer, warp 1 MMA issuer, warps 2..17 consumers: TMEM lane = query row, four threads per
// row (warps w, w + 4, w + 8, w + 12 read the same lane quadrant).  The maxima and Newton sweeps walk 256-key tiles
// (N = 256 MMA groups into two 256-column accumulators, a thread scanning 64 columns), the output sweep 128-key
// tiles (two 128-column S accumulators beside the O accumulator, a thread scanning 32 columns); at the end of a
// sweep the four threads of a row swap their partial sums through shared memory.  The number of Newton sweeps is decided by the
// consumers; they publish "all rows converged" through shared memory and a control mbarrier that every role
// waits on between sweeps.  Every wait is bounded (see sm100_ptx.cuh); on expiry the CTA flags the call's status
// word and leaves.
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace entmax {

namespace {

using namespace sm100;

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}

constexpr int TM = 128;            // query rows per item = TMEM lanes
constexpr int TN = 128;            // keys per K/V tile of the output sweep
constexpr int TW = 2 * TN;         // keys per K tile of every other sweep (two tile slots, one MMA group of N = 256)
constexpr int kConsGroups = 4;                       // threads per query row
constexpr int kConsWarps = 4 * kConsGroups;           // four TMEM lane quadrants each
constexpr int kThreadsT = (3 + kConsWarps) * 32;      // TMA warp, score MMA warp, the consumer warps, P V MMA warp
constexpr int kPvWarp = 2 + kConsWarps;
constexpr int kMaxSweeps = 48;     // 1 max sweep + at most 46 Newton sweeps + the output sweep
// Sampled start: long rows first solve Eq. 1's threshold on every kTileSampleStride-th key (sweeps an eighth as long),
// each sampled key counted kTileSampleStride times, so that the sample's threshold estimates the row's; the full-row
// Newton iteration starts from it instead of from y_max - 1 and needs no y_max sweep.  An estimate past the root costs
// nothing more than one from before it: F = S^(1/e) - 1 is convex and decreasing, so the first Newton step from
// there lands at or before the root and the iteration goes on from the left (steps from the left never pass it).
constexpr int kTileSampleStride = 8;
constexpr int kSampleMinTiles = 16;    // K tiles a Q tile must see for the sampled start to pay
constexpr int kSampleSweepCap = 12;    // sampled sweeps at most
constexpr float kSampleTol = 1e-2f;    // the sampled iteration stops at a step of this size, relative to |tau|
// Mass sum_j p_ij at the threshold a sweep used, minus 1.  Within kNearMass before a Newton step: the step squares the
// error, so the next sweep can be an output sweep.  Within kOutputMass in an output sweep: its O is the result (P is
// rounded to bf16, 2^-9 relative, anyway), and the step its sums give makes the stored threshold exact to fp32.
constexpr float kNearMass = 5e-2f, kOutputMass = 1e-3f;
enum SweepKind : int { kSampleMax = 0, kSampleNewton = 1, kFullMax = 2, kFullNewton = 3, kOutput = 4 };
constexpr int kPBytes = TM * TN * 2;

template <int HD>
struct TCfg {
  static constexpr int kHalves = HD / 64;
  static constexpr int kQBytes = TM * HD * 2;
  static constexpr int kKBytes = TN * HD * 2;      // also the size of a V tile
  static constexpr int kBarBytes = 384;
  static constexpr int kXchgBytes = 2 * kConsGroups * TM * 8;   // one float2 per (exchange parity, thread of a row, row)
  static constexpr int kStages = HD == 64 ? 4 : 2;   // K/V ring depth of the output sweep: what fits beside Q and P
  static constexpr int kSmemBytes = kQBytes + kStages * 2 * kKBytes + kPBytes + 1024 + kBarBytes + kXchgBytes;
  static constexpr int kTmemO = 2 * TN;            // first TMEM column of the O accumulator
};

struct TileArgsK {
  int B, H, N;
  int causal;
  int expo_class;
  float expo;
  float alpha_m1;
  float sm_scale;
  const float* scale;        // [H, N] (scale_sb = 0) or [B, H, N] (scale_sb = H*N)
  const float* alibi;        // [H] ALiBi slopes or nullptr (causal problems only)
  long long scale_sb;
  const int32_t* tile_list;  // ids of the Q tiles to process: bh * tiles_per_head + tile
  const int32_t* tile_count;
  int32_t* work_counter;     // next position of tile_list to hand out (zero on entry)
  const int32_t* row_cnt;    // -2 marks the rows to write
  int32_t* dense_cnt;        // [B*H*N][2]: support size each of a row's two threads counted (written rows only)
  void* o;                   // bf16 [B,H,N,D]
  float* tau;
  int64_t sb, sh, sn;
  int32_t* status;
  int tiles_per_head;
};

// S = Q K^T: A, B bf16 K-major, fp32 accumulate, M = 128, N = TN (output sweep) or TW (the other sweeps)
__host__ __device__ constexpr uint32_t idesc_qk(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
}
// O += P V: A = P K-major, B = V with N (head dim) contiguous ("MN-major", bit 16), M = 128, N = HD
template <int HD>
__host__ __device__ constexpr uint32_t idesc_pv() {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(HD >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
}
// Descriptor words of the V tile as an N-major operand with 128-byte swizzle: a swizzle atom is 64
// head-dim elements (one 128-byte row) by 8 keys; atoms repeat every 1024 bytes along the keys
// (stride-dimension offset) and, for head_dim 128, every TN*128 bytes along the head dimension
// (leading-dimension offset: the second 64-column block of the tile).
__device__ __forceinline__ uint32_t v_desc_lo(uint32_t saddr) {
  return ((saddr & 0x3FFFFu) >> 4) | ((uint32_t)((TN * 128) >> 4) << 16);
}

template <int HD, int EC>
__global__ void __launch_bounds__(kThreadsT, 1) tile_fwd_kernel(const __grid_constant__ CUtensorMap map_q,
                                                               const __grid_constant__ CUtensorMap map_k,
                                                               const __grid_constant__ CUtensorMap map_v,
                                                               const __grid_constant__ CUtensorMap map_ks,
                                                               const TileArgsK a) {
  using C = TCfg<HD>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_smem = sbase;
  // tile slots: the output sweep keeps 128-key K tiles in the first half and V tiles in the second, (K, V) of a
  // stage arriving on the stage's barrier; the other sweeps keep one 256-key K tile per stage in two adjacent slots
  const uint32_t k_smem = q_smem + C::kQBytes;                       // [2 * C::kStages] tile slots
  const uint32_t v_smem = k_smem + C::kStages * C::kKBytes;            // = slot C::kStages
  const uint32_t p_smem = v_smem + C::kStages * C::kKBytes;            // P tile, A-operand layout
  const uint32_t bars = p_smem + kPBytes;
  const uint32_t q_full = bars, q_empty = bars + 8;
  const uint32_t kv_full = bars + 16;                                 // [C::kStages]
  const uint32_t kv_empty = kv_full + 8 * C::kStages;                   // [C::kStages]
  const uint32_t s_full = kv_empty + 8 * C::kStages;                    // [2]
  const uint32_t s_empty = s_full + 16;                               // [2]
  const uint32_t p_full = s_empty + 16, p_empty = p_full + 8;
  const uint32_t o_full = p_empty + 8, o_empty = o_full + 8;
  const uint32_t ctl = o_empty + 8;                                   // the consumers' vote on a sweep is in
  const uint32_t done_word = ctl + 8;                                 // uint32 [3]
  const uint32_t x_bar = done_word + 16;                              // partial sums of a sweep are in shared memory
  const uint32_t tmem_slot = x_bar + 8;
  const uint32_t abort_flag = tmem_slot + 4;
  const uint32_t drain_bar = tmem_slot + 8;                           // teardown: every MMA issued so far has finished
  const uint32_t drain_fail = drain_bar + 8;                          // uint32: a teardown wait ran out as well
  const uint32_t w_full = drain_fail + 8;                             // [2] a work item has been published
  const uint32_t w_empty = w_full + 16;                               // [2] ... and read by the MMA issuer and every consumer warp
  const uint32_t w_item = w_empty + 16;                               // int32 [2]: tile id, -1 = no more work
  const uint32_t v_full = w_item + 8;                                 // [C::kStages] output sweep: V tiles on barriers
  const uint32_t v_empty = v_full + 8 * C::kStages;                     // [C::kStages]   of their own (see the producer)
  const uint32_t drain_bar_pv = v_empty + 8 * C::kStages;               // teardown, the P V issuer's contractions
  const uint32_t xchg = bars + C::kBarBytes;                          // float2 [2][kConsGroups][TM]
  static_assert(8 * (2 + 4 * C::kStages + 4 + 4 + 1) + 16 + 8 + 8 + 16 + 40 + 8 <= C::kBarBytes, "barrier area");

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int n_tiles = *a.tile_count;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    mbar_init(q_empty, 1);
    for (int t = 0; t < C::kStages; ++t) {
      mbar_init(kv_full + 8 * t, 1);
      mbar_init(kv_empty + 8 * t, 1);
      mbar_init(v_full + 8 * t, 1);
      mbar_init(v_empty + 8 * t, 1);
    }
    for (int t = 0; t < 2; ++t) {
      mbar_init(s_full + 8 * t, 1);
      mbar_init(s_empty + 8 * t, kConsWarps);
    }
    mbar_init(p_full, kConsWarps);
    mbar_init(p_empty, 1);
    mbar_init(o_full, 1);
    mbar_init(o_empty, kConsWarps);
    mbar_init(ctl, kConsWarps + 1);                     // the consumer warps' votes and the P V issuer keeping in step
    mbar_init(x_bar, kConsWarps);
    for (int t = 0; t < 3; ++t) sts_u32(done_word + 4 * t, 3u);
    mbar_init(drain_bar, 1);
    mbar_init(drain_bar_pv, 1);
    for (int t = 0; t < 2; ++t) {
      mbar_init(w_full + 8 * t, 1);
      mbar_init(w_empty + 8 * t, 2 + kConsWarps);   // the two MMA issuers + the consumer warps
    }
    sts_u32(drain_fail, 0u);
    sts_u32(abort_flag, 0u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = lds_u32(tmem_slot);

  // Sweeps of an item.  Without the sampled start: sweep 0 finds the row maxima, then Newton sweeps until the
  // consumers report that every row has converged (or the cap is reached), then the output sweep.  With it: a maxima
  // sweep and Newton sweeps over the sampled keys first, then Newton sweeps over all keys from the sample's
  // threshold, then the output sweep.  All roles evaluate this the same way, once per sweep, after the vote is in.
  auto item_tiles = [&](int tile) -> int {
    const int row0 = tile * TM;
    if (!a.causal) return (a.N + TN - 1) / TN;
    int last_row = row0 + TM - 1;
    if (last_row > a.N - 1) last_row = a.N - 1;
    return last_row / TN + 1;
  };
  // sampled K tiles of an item (0: no sampled start)
  auto item_sample_tiles = [&](int tile) -> int {
    if (a.expo < 1.0f || item_tiles(tile) < kSampleMinTiles) return 0;
    int last_row = tile * TM + TM - 1;
    if (last_row > a.N - 1) last_row = a.N - 1;
    const int n_vis = a.causal ? last_row + 1 : a.N;
    int groups = (n_vis + kTileSampleStride - 1) / kTileSampleStride;
    if (groups > a.N / kTileSampleStride) groups = a.N / kTileSampleStride;
    return (groups + TN - 1) / TN;
  };
  // The consumers' vote on sweep s - 1: bit 0 = every row of the tile has its final threshold, bit 1 = every row's mass
  // was within kNearMass of 1 before its last step.  An output sweep is started as soon as every row is near: it also
  // takes the Newton sums, and if they show every row's mass within kOutputMass of 1, its O is the result (the stored
  // threshold takes the last step too); otherwise the iteration goes on and another output sweep follows.
  auto prev_vote = [&](int s) -> uint32_t { return s >= 1 ? lds_u32(done_word + 4 * ((s - 1) % 3)) : 0u; };
  auto sweep_kind = [&](int s, int& phase, int& n_full) -> int {
    const uint32_t vote = prev_vote(s);
    const bool prev_done = (vote & 1u) != 0u;
    if (phase == 0) {
      if (s == 0) return kSampleMax;
      if ((prev_done && s >= 2) || s >= kSampleSweepCap) {
        phase = 1;
        n_full = 1;
        return kFullNewton;
      }
      return kSampleNewton;
    }
    if (s == 0) return kFullMax;
    if (s >= kMaxSweeps - 1 || (vote != 0u && n_full >= 1)) return kOutput;
    ++n_full;
    return kFullNewton;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    // (the whole warp runs the control flow, one elected lane issues the copies: see the MMA issuer)
    {
      int slot = 0;
      uint32_t kvbits = 0 /* bit x: times barrier pair x has been armed, mod 2 */, vbits = 0, qphase = 0, cphase = 0,
               wphase = 0;
      bool alive = true;
      auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
      };
      while (alive) {
        // items are handed out from a shared counter, in the list's order (longest first on causal problems), so
        // that the CTAs finish together whatever the Q tiles' lengths and sweep counts are
        alive = wait_all(w_empty + 8 * slot, wphase ^ 1u);
        if (!alive) break;
        int id = 0;
        if (lane == 0) {
          const int it = atomicAdd(a.work_counter, 1);
          id = it < n_tiles ? a.tile_list[it] : -1;
          sts_u32(w_item + 4 * slot, (uint32_t)id);
          mbar_arrive(w_full + 8 * slot);
        }
        id = __shfl_sync(0xffffffffu, id, 0);
        if (++slot == 2) { slot = 0; wphase ^= 1u; }
        if (id < 0) break;
        const int bh = id / a.tiles_per_head, tile = id - bh * a.tiles_per_head;
        const int b = bh / a.H, h = bh - b * a.H;
        const int tiles = item_tiles(tile), stiles = item_sample_tiles(tile);
        int phase = stiles > 0 ? 0 : 1, n_full = 0;
        alive = wait_all(q_empty, qphase ^ 1u);
        if (!alive) break;
        if (elect_one()) {
          mbar_expect_tx(q_full, C::kQBytes);
          for (int hf = 0; hf < C::kHalves; ++hf)
            tma_load_4d(q_smem + hf * (TM * 128), &map_q, q_full, hf * 64, tile * TM, h, b);
        }
        __syncwarp();
        qphase ^= 1u;
        bool was_output = false;
        for (int s = 0; alive; ++s) {
          if (s > 0) {
            alive = wait_all(ctl, cphase);
            cphase ^= 1u;
            if (!alive) break;
            // an output sweep whose threshold the vote confirms ends the item
            if (was_output && __shfl_sync(0xffffffffu, (int)(prev_vote(s) & 1u), 0)) break;
          }
          int kind = sweep_kind(s, phase, n_full);
          kind = __shfl_sync(0xffffffffu, kind, 0);
          phase = __shfl_sync(0xffffffffu, phase, 0);
          n_full = __shfl_sync(0xffffffffu, n_full, 0);
          const bool output = kind == kOutput, smp = kind <= kSampleNewton;
          was_output = output;
          // the output sweep walks 128-key tiles; every other sweep walks 256-key tiles, two tile slots to a stage,
          // rows 128.. of a 64-column block right behind rows 0..127
          const int nt = output ? tiles : ((smp ? stiles : tiles) + 1) / 2;
          const int ring = C::kStages;   // every sweep starts at stage 0
          int stage = 0;
          if (output) {
            // K and V tiles on barriers of their own, K one tile ahead of V: a K slot is free as soon as the scores
            // of the tile before last have been formed, a V slot only after that tile's P V -- on one barrier the
            // next K tile was asked for a whole contraction late and the issuer waited out the copy on every tile
            int ks = 0, vs = 0;
            auto load_kv = [&](const CUtensorMap* map, uint32_t full, uint32_t empty, uint32_t smem, uint32_t& bits,
                               int& st, int t) -> bool {
              if (!wait_all(empty + 8 * st, ((bits >> st) & 1u) ^ 1u)) return false;
              bits ^= 1u << st;
              if (elect_one()) {
                mbar_expect_tx(full + 8 * st, C::kKBytes);
                for (int hf = 0; hf < C::kHalves; ++hf)
                  tma_load_4d(smem + st * C::kKBytes + hf * (TN * 128), map, full + 8 * st, hf * 64, t * TN, h, b);
              }
              __syncwarp();
              if (++st == ring) st = 0;
              return true;
            };
            alive = load_kv(&map_k, kv_full, kv_empty, k_smem, kvbits, ks, 0);
            for (int t = 0; t < nt && alive; ++t) {
              if (t + 1 < nt) alive = load_kv(&map_k, kv_full, kv_empty, k_smem, kvbits, ks, t + 1);
              if (alive) alive = load_kv(&map_v, v_full, v_empty, v_smem, vbits, vs, t);
            }
            continue;
          }
          for (int t = 0; t < nt && alive; ++t) {
            alive = wait_all(kv_empty + 8 * stage, ((kvbits >> stage) & 1u) ^ 1u);
            if (!alive) break;
            kvbits ^= 1u << stage;
            if (elect_one()) {
              mbar_expect_tx(kv_full + 8 * stage, 2 * C::kKBytes);
              for (int hf = 0; hf < C::kHalves; ++hf) {
#pragma unroll
                for (int rh = 0; rh < 2; ++rh) {
                  const uint32_t dst = k_smem + stage * 2 * C::kKBytes + hf * (TW * 128) + rh * (TN * 128);
                  if (smp) tma_load_5d(dst, &map_ks, kv_full + 8 * stage, hf * 64, 0, t * TW + rh * TN, h, b);
                  else tma_load_4d(dst, &map_k, kv_full + 8 * stage, hf * 64, t * TW + rh * TN, h, b);
                }
              }
            }
            __syncwarp();
            if (++stage == ring) stage = 0;
          }
        }
      }
      if (!alive && lane == 0) {
        // a wait ran out somewhere in the CTA: the copies this warp armed barriers for must land before shared
        // memory goes away (the phase armed last has the parity opposite to the arm count's)
        bool ok = mbar_drain(q_full, qphase ^ 1u);
        for (int st = 0; st < C::kStages; ++st) ok &= mbar_drain(kv_full + 8 * st, ((kvbits >> st) & 1u) ^ 1u);
        for (int st = 0; st < C::kStages; ++st) ok &= mbar_drain(v_full + 8 * st, ((vbits >> st) & 1u) ^ 1u);
        if (!ok) sts_u32(drain_fail, 1u);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (scores)
    // The whole warp runs this role's control flow (waits are voted on, values read from shared memory are
    // broadcast), so that descriptors, addresses and counters are warp-uniform; one elected lane issues the tensor
    // core instructions.  A single lane inside a divergent branch would compete for issue slots with the consumer
    // warps of its scheduler for every address calculation of every MMA.
    {
      constexpr uint32_t id_qk = idesc_qk(TN), id_qk_wide = idesc_qk(TW);
      const uint64_t hi = (uint64_t)kDescHi << 32;
      const uint64_t q_desc = hi | smem_desc_lo(q_smem), k_desc = hi | smem_desc_lo(k_smem);
      uint32_t kvbits = 0 /* bit x: phase of barrier pair x to wait for */, qphase = 0, cphase = 0, sphase[2] = {0, 0},
               ophase = 0;
      int sbuf = 0, slot = 0;
      uint32_t wphase = 0;
      bool alive = true;
      auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
      };
      while (alive) {
        alive = wait_all(w_full + 8 * slot, wphase);
        if (!alive) break;
        const int id = __shfl_sync(0xffffffffu, (int)lds_u32(w_item + 4 * slot), 0);
        __syncwarp();
        if (lane == 0) mbar_arrive(w_empty + 8 * slot);
        if (++slot == 2) { slot = 0; wphase ^= 1u; }
        if (id < 0) break;
        const int tile = id % a.tiles_per_head;
        const int tiles = item_tiles(tile), stiles = item_sample_tiles(tile);
        int phase = stiles > 0 ? 0 : 1, n_full = 0;
        alive = wait_all(q_full, qphase);
        qphase ^= 1u;
        if (!alive) break;
        // the previous item's O must have been read before this item's MMAs start: its columns are the second wide
        // accumulator of the sweeps that come first, and the O accumulator of the output sweep
        alive = wait_all(o_empty, ophase ^ 1u);
        ophase ^= 1u;
        if (!alive) break;
        bool was_output = false;
        for (int s = 0; alive; ++s) {
          if (s > 0) {
            alive = wait_all(ctl, cphase);
            cphase ^= 1u;
            if (!alive) break;
            if (was_output && __shfl_sync(0xffffffffu, (int)(prev_vote(s) & 1u), 0)) break;
          }
          int kind = sweep_kind(s, phase, n_full);
          kind = __shfl_sync(0xffffffffu, kind, 0);
          phase = __shfl_sync(0xffffffffu, phase, 0);
          n_full = __shfl_sync(0xffffffffu, n_full, 0);
          const bool output = kind == kOutput;
          was_output = output;
          const int nt = output ? tiles : ((kind <= kSampleNewton ? stiles : tiles) + 1) / 2;
          const int ring = C::kStages;   // every sweep starts at stage 0
          int stage = 0;
          // S = Q K^T of the next K tile into the accumulator the consumers have handed back: 128 keys and columns
          // in the output sweep, 256 in the others (which do not use the O accumulator's columns for O)
          auto issue_qk = [&]() -> bool {
            bool ok = wait_all(kv_full + 8 * stage, (kvbits >> stage) & 1u);
            if (ok) ok = wait_all(s_empty + 8 * sbuf, sphase[sbuf] ^ 1u);
            if (!ok) return false;
            kvbits ^= 1u << stage;
            sphase[sbuf] ^= 1u;
            tc_fence_after();
            if (output) {
              const uint64_t b_desc = k_desc + (uint64_t)(stage * (C::kKBytes >> 4));
              const uint32_t d_tmem = tmem_base + sbuf * TN;
              if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                  const uint32_t a_off = (kk >> 2) * ((TM * 128) >> 4) + (kk & 3) * 2;
                  const uint32_t b_off = (kk >> 2) * ((TN * 128) >> 4) + (kk & 3) * 2;
                  umma_bf16_desc(d_tmem, q_desc + a_off, b_desc + b_off, id_qk, kk > 0 ? 1u : 0u);
                }
                umma_commit(s_full + 8 * sbuf);
                umma_commit(kv_empty + 8 * stage);   // the K slot is free once these scores are formed
              }
            } else {
              const uint64_t b_desc = k_desc + (uint64_t)(stage * (2 * C::kKBytes >> 4));
              const uint32_t d_tmem = tmem_base + sbuf * TW;
              if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                  const uint32_t a_off = (kk >> 2) * ((TM * 128) >> 4) + (kk & 3) * 2;
                  const uint32_t b_off = (kk >> 2) * ((TW * 128) >> 4) + (kk & 3) * 2;
                  umma_bf16_desc(d_tmem, q_desc + a_off, b_desc + b_off, id_qk_wide, kk > 0 ? 1u : 0u);
                }
                umma_commit(s_full + 8 * sbuf);
              }
            }
            __syncwarp();
            sbuf ^= 1;
            return true;
          };
          if (!output) {
            for (int t = 0; t < nt && alive; ++t) {
              alive = issue_qk();
              if (!alive) break;
              if (elect_one()) umma_commit(kv_empty + 8 * stage);
              __syncwarp();
              if (++stage == ring) stage = 0;
            }
          } else {
            // output sweep: the scores run ahead of the consumers as far as the two accumulators allow; O += P V is
            // issued by a warp of its own, so that neither stream of contractions waits for the other's barriers and
            // each issuer's instruction count per tile is halved (the issuers compete for issue slots with the
            // consumer warps of their schedulers: a tile's sixteen MMAs from one warp took ~2200 cycles)
            for (int t = 0; t < nt && alive; ++t) {
              alive = issue_qk();
              if (!alive) break;
              if (++stage == ring) stage = 0;
            }
          }
        }
        if (elect_one()) umma_commit(q_empty);
        __syncwarp();
      }
      if (!alive && lane == 0) {
        // the tensor core must be done with shared memory and TMEM before they are released
        umma_commit(drain_bar);
        if (!mbar_drain(drain_bar, 0u)) sts_u32(drain_fail, 1u);
      }
    }
  } else if (warp == kPvWarp) {
    // ------------------------------------------------------------------ P V issuer (output sweeps only)
    // Follows the sweeps of every item like the other roles (warp-wide control flow, one elected lane issuing) and
    // arrives on the control barrier once per sweep, so that it can never fall a whole sweep behind the consumers.
    {
      constexpr uint32_t id_pv = idesc_pv<HD>();
      const uint64_t hi = (uint64_t)kDescHi << 32;
      const uint64_t p_desc = hi | smem_desc_lo(p_smem), v_desc = hi | v_desc_lo(v_smem);
      uint32_t vbits = 0 /* bit x: phase of V barrier pair x to wait for */, cphase = 0, pphase = 0, wphase = 0;
      int slot = 0;
      bool alive = true;
      auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
      };
      while (alive) {
        alive = wait_all(w_full + 8 * slot, wphase);
        if (!alive) break;
        const int id = __shfl_sync(0xffffffffu, (int)lds_u32(w_item + 4 * slot), 0);
        __syncwarp();
        if (lane == 0) mbar_arrive(w_empty + 8 * slot);
        if (++slot == 2) { slot = 0; wphase ^= 1u; }
        if (id < 0) break;
        const int tile = id % a.tiles_per_head;
        const int tiles = item_tiles(tile), stiles = item_sample_tiles(tile);
        int phase = stiles > 0 ? 0 : 1, n_full = 0;
        bool was_output = false;
        for (int s = 0; alive; ++s) {
          if (s > 0) {
            alive = wait_all(ctl, cphase);
            cphase ^= 1u;
            if (!alive) break;
            if (was_output && __shfl_sync(0xffffffffu, (int)(prev_vote(s) & 1u), 0)) break;
          }
          int kind = sweep_kind(s, phase, n_full);
          kind = __shfl_sync(0xffffffffu, kind, 0);
          phase = __shfl_sync(0xffffffffu, phase, 0);
          n_full = __shfl_sync(0xffffffffu, n_full, 0);
          was_output = kind == kOutput;
          if (was_output) {
            int vstage = 0;   // every sweep starts at stage 0
            for (int t = 0; t < tiles && alive; ++t) {
              // O += P V for this tile once the consumers have written P and the V tile has landed
              alive = wait_all(p_full, pphase);
              pphase ^= 1u;
              if (alive) alive = wait_all(v_full + 8 * vstage, (vbits >> vstage) & 1u);
              if (!alive) break;
              vbits ^= 1u << vstage;
              tc_fence_after();
              const uint64_t vb_desc = v_desc + (uint64_t)(vstage * (C::kKBytes >> 4));
              if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < TN / 16; ++kk) {
                  const uint32_t a_off = (kk >> 2) * ((TM * 128) >> 4) + (kk & 3) * 2;   // 64 keys per 128-byte row
                  const uint32_t b_off = kk * ((16 * 128) >> 4);                           // 16 keys = 16 rows of 128 B
                  umma_bf16_desc(tmem_base + C::kTmemO, p_desc + a_off, vb_desc + b_off, id_pv,
                                 (t > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(p_empty);
                umma_commit(v_empty + 8 * vstage);
                if (t == tiles - 1) umma_commit(o_full);
              }
              __syncwarp();
              if (++vstage == C::kStages) vstage = 0;
            }
            if (!alive) break;
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(ctl);
        }
      }
      if (!alive && lane == 0) {
        // this warp's contractions must be done with shared memory and TMEM before they are released
        umma_commit(drain_bar_pv);
        if (!mbar_drain(drain_bar_pv, 0u)) sts_u32(drain_fail, 1u);
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers: four threads per query row
    // (warps w, w + 4, w + 8, w + 12 share a TMEM lane quadrant; `quarter` picks the 32 of a tile's 128 columns a
    // thread scans).  A thread's share of a tile is one TMEM load; the accumulator goes back to the MMA issuer as
    // soon as the load has landed in registers.
    const int quad = warp & 3;
    const int quarter = (warp - 2) >> 2;
    const int row_local = quad * 32 + lane;
    const uint32_t taddr_row = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint32_t sphase[2] = {0, 0}, pphase = 0, ophase = 0, cphase = 0, xphase = 0, wphase = 0;
    int sbuf = 0, slot = 0;
    bool alive = true;
    // the four threads of a row swap partial results through shared memory: slot [exchange parity][quarter][row]; all
    // four then add the same four numbers in the same order
    auto swap4 = [&](float x0, float x1, float (&r0)[4], float (&r1)[4]) -> bool {
      const uint32_t base = xchg + xphase * (uint32_t)(kConsGroups * TM * 8);
      const uint32_t mine = base + (uint32_t)(quarter * TM + row_local) * 8u;
      sts_u32(mine, __float_as_uint(x0));
      sts_u32(mine + 4, __float_as_uint(x1));
      __syncwarp();
      if (lane == 0) mbar_arrive(x_bar);
      const bool ok = __all_sync(0xffffffffu, mbar_wait(x_bar, xphase, abort_flag));
      xphase ^= 1u;
      if (!ok) return false;
#pragma unroll
      for (int g = 0; g < kConsGroups; ++g) {
        r0[g] = __uint_as_float(lds_u32(base + (uint32_t)(g * TM + row_local) * 8u));
        r1[g] = __uint_as_float(lds_u32(base + (uint32_t)(g * TM + row_local) * 8u + 4u));
      }
      return true;
    };
    while (alive) {
      alive = __all_sync(0xffffffffu, mbar_wait(w_full + 8 * slot, wphase, abort_flag));
      if (!alive) break;
      const int id = (int)lds_u32(w_item + 4 * slot);
      __syncwarp();
      if (lane == 0) mbar_arrive(w_empty + 8 * slot);
      if (++slot == 2) { slot = 0; wphase ^= 1u; }
      if (id < 0) break;
      const int bh = id / a.tiles_per_head, tile = id - bh * a.tiles_per_head;
      const int b = bh / a.H, h = bh - b * a.H;
      const int tiles = item_tiles(tile), stiles = item_sample_tiles(tile);
      int phase = stiles > 0 ? 0 : 1, n_full = 0, n_smp = 0;
      const int i = tile * TM + row_local;
      const bool valid = i < a.N;
      const size_t grow = (size_t)bh * a.N + (valid ? i : 0);
      const int lim = a.causal ? i : a.N - 1;
      // last sampled column (key kTileSampleStride * column) this row may look at
      int glim = lim / kTileSampleStride;
      if (glim > a.N / kTileSampleStride - 1) glim = a.N / kTileSampleStride - 1;
      const float ra = valid ? a.alpha_m1 * (a.scale[(size_t)b * a.scale_sb + (size_t)h * a.N + i] * a.sm_scale) : 0.f;
      const float slope = a.alibi ? a.alibi[h] / a.sm_scale : 0.f;   // bias in accumulator units
      float tau = 0.f, ymax = -INFINITY;
      TauIter it_tau = {0.f, 0.f, 0.f};
      bool done = !valid, was_output = false;
      int n_supp_out = 0;
      for (int s = 0; alive; ++s) {
        if (s > 0) {
          alive = __all_sync(0xffffffffu, mbar_wait(ctl, cphase, abort_flag));
          cphase ^= 1u;
          if (!alive) break;
          if (was_output && (prev_vote(s) & 1u)) {
            // ---- the vote confirms the thresholds the last output sweep used: its O is the result
            tc_fence_after();
            const bool write = valid && a.row_cnt[grow] == -2;
            __nv_bfloat16* orow =
                reinterpret_cast<__nv_bfloat16*>(a.o) + (size_t)b * a.sb + (size_t)h * a.sh + (size_t)i * a.sn;
            for (int c = quarter; c < HD / 32; c += kConsGroups) {
              float va[32];
              tmem_ld32(taddr_row + C::kTmemO + c * 32, va);
              tmem_ld_wait();
              if (write) {
#pragma unroll
                for (int u8 = 0; u8 < 4; ++u8) {
                  uint32_t w[4];
#pragma unroll
                  for (int e2 = 0; e2 < 4; ++e2) {
                    const __nv_bfloat162 hh = __floats2bfloat162_rn(va[u8 * 8 + e2 * 2], va[u8 * 8 + e2 * 2 + 1]);
                    w[e2] = *reinterpret_cast<const uint32_t*>(&hh);
                  }
                  *reinterpret_cast<uint4*>(orow + c * 32 + u8 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                }
              }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(o_empty);
            // the row's support size, as two halves (keys of the tile's first / second 64 columns)
            float n4[4], unused[4];
            alive = swap4((float)n_supp_out, 0.f, n4, unused);
            if (!alive) break;
            if (write && quarter == 0) a.tau[grow] = tau;
            if (write && (quarter & 1) == 0) a.dense_cnt[grow * 2 + (quarter >> 1)] = (int)(n4[quarter] + n4[quarter + 1]);
            if (a.status && threadIdx.x == 64) {
              // diagnostics: full-length sweeps spent (y_max sweep if any, Newton sweeps, output sweep; the sampled
              // sweeps, an eighth as long, are not counted) and tiles processed
              atomicAdd(a.status + ENTMAX_ATTN_STATUS_TILE_SWEEPS, s - n_smp);
              atomicAdd(a.status + ENTMAX_ATTN_STATUS_TILES, 1);
            }
            break;
          }
        }
        const int kind = sweep_kind(s, phase, n_full);
        const bool output = kind == kOutput, smp = kind <= kSampleNewton;
        was_output = output;
        const bool find_max = kind == kSampleMax || kind == kFullMax;
        // the output sweep walks 128-key tiles (a thread scans 32 columns); every other sweep walks 256-key tiles
        // (two accumulators of 256 columns; a thread scans 64 columns as two chunks)
        const int nt = output ? tiles : ((smp ? stiles : tiles) + 1) / 2;
        const int lim_c = smp ? glim : lim;            // in the column space of this sweep
        const float slope_c = smp ? slope * (float)kTileSampleStride : slope;
        if (kind == kFullNewton && n_full == 1 && stiles > 0) done = !valid;   // the full-row iteration starts here
        n_smp += smp ? 1 : 0;
        float s0 = 0.f, s1 = 0.f;
        int n_supp = 0;   // output sweep: keys of this thread's columns with p > 0
        // one 32-column chunk of a maxima or Newton sweep
        auto scan_chunk = [&](float (&va)[32], const int col0) {
          if (slope != 0.f) {
            // bias m_h (key - i) in accumulator units; a sampled column stands for key kTileSampleStride * column
#pragma unroll
            for (int u = 0; u < 32; ++u) va[u] = fmaf(slope_c, (float)(col0 + u), va[u]) - slope * (float)i;
          }
          // columns past the row's last visible key only occur in the tiles at the causal diagonal / the tail
          const bool edge = col0 + 31 > lim_c;
          if (find_max) {
            // y_max over the visible keys
            float m[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int u = 0; u < 32; ++u) {
              const float yv = ra * va[u];
              m[u & 3] = fmaxf(m[u & 3], (!edge || col0 + u <= lim_c) ? yv : -INFINITY);
            }
            ymax = fmaxf(ymax, fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3])));
          } else {
            if (EC != kExpoGeneral && !edge) {
              // the bulk of a Newton sweep.  What limits it is the ALU pipe (half the FMA pipe's rate), so per
              // element one clamp there and everything else as FMA-pipe work: y = a acc - tau, its powers fused
              // into the running sums (four partial sums per total)
              float p0[4] = {0.f, 0.f, 0.f, 0.f}, p1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int u = 0; u < 32; ++u) {
                const float m = fmaxf(fmaf(ra, va[u], -tau), 0.f);
                if constexpr (EC == kExpo2) {
                  p0[u & 3] = fmaf(m, m, p0[u & 3]);
                  p1[u & 3] += m;
                } else if constexpr (EC == kExpo4) {
                  const float t2 = m * m;
                  p0[u & 3] = fmaf(t2, t2, p0[u & 3]);
                  p1[u & 3] = fmaf(t2, m, p1[u & 3]);
                } else {
                  p0[u & 3] += m;
                  p1[u & 3] += positive_indicator(m);
                }
              }
              s0 += (p0[0] + p0[1]) + (p0[2] + p0[3]);
              s1 += (p1[0] + p1[1]) + (p1[2] + p1[3]);
            } else {
              // four independent partial sums each, so that the additions do not form one serial chain
              float p0[4] = {0.f, 0.f, 0.f, 0.f}, p1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int u = 0; u < 32; ++u) {
                const float yr = fmaf(ra, va[u], -tau);
                const bool ok = yr > 0.f && (!edge || col0 + u <= lim_c);
                float ye, ye1;
                pow_pair_c<EC>(ok ? yr : 0.f, ok, a.expo, ye, ye1);
                p0[u & 3] += ye;
                p1[u & 3] += ye1;
              }
              s0 += (p0[0] + p0[1]) + (p0[2] + p0[3]);
              s1 += (p1[0] + p1[1]) + (p1[2] + p1[3]);
            }
          }
        };
        for (int t = 0; t < nt && alive; ++t) {
          alive = __all_sync(0xffffffffu, mbar_wait(s_full + 8 * sbuf, sphase[sbuf], abort_flag));
          if (!alive) break;
          sphase[sbuf] ^= 1u;
          tc_fence_after();
          if (!output) {
            float va0[32], va1[32];
            tmem_ld32(taddr_row + sbuf * TW + quarter * 64, va0);
            tmem_ld32(taddr_row + sbuf * TW + quarter * 64 + 32, va1);
            tmem_ld_wait();
            // the scores are in registers: the accumulator can take the tile after next
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(s_empty + 8 * sbuf);
            sbuf ^= 1;
            scan_chunk(va0, t * TW + quarter * 64);
            scan_chunk(va1, t * TW + quarter * 64 + 32);
            continue;
          }
          float va[32];
          tmem_ld32(taddr_row + sbuf * TN + quarter * 32, va);
          tmem_ld_wait();
          // the scores are in registers: the accumulator can take the tile after next
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(s_empty + 8 * sbuf);
          sbuf ^= 1;
          const int col0 = t * TN + quarter * 32;
          if (slope != 0.f) {
            // bias m_h (key - i) in accumulator units
#pragma unroll
            for (int u = 0; u < 32; ++u) va[u] = fmaf(slope, (float)(col0 + u), va[u]) - slope * (float)i;
          }
          // columns past the row's last visible key only occur in the tiles at the causal diagonal / the tail
          const bool edge = col0 + 31 > lim;
          {
            // P -> bf16, formed in registers while the tensor core still reads the previous P tile
            uint32_t w[16];
            if (EC != kExpoGeneral && !edge) {
              // as in the Newton sweeps: one ALU-pipe clamp per element, the rest on the FMA pipe (the count of
              // positive entries too: an indicator formed by a saturating multiply).  Rows past the end of the
              // sequence have a = 0, tau = 0: all zero.
              float cnt[4] = {0.f, 0.f, 0.f, 0.f}, q0[4] = {0.f, 0.f, 0.f, 0.f}, q1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int e2 = 0; e2 < 16; ++e2) {
                float pv[2];
#pragma unroll
                for (int z = 0; z < 2; ++z) {
                  const float m = fmaxf(fmaf(ra, va[e2 * 2 + z], -tau), 0.f);
                  const float ind = positive_indicator(m);
                  float ye1;
                  if constexpr (EC == kExpo2) { ye1 = m; pv[z] = m * m; }
                  else if constexpr (EC == kExpo4) { const float t2 = m * m; ye1 = t2 * m; pv[z] = t2 * t2; }
                  else { ye1 = ind; pv[z] = m; }
                  cnt[(e2 * 2 + z) & 3] += ind;
                  // the Newton sums at this threshold too: they decide whether this sweep's O is the result
                  q0[(e2 * 2 + z) & 3] += pv[z];
                  q1[(e2 * 2 + z) & 3] += ye1;
                }
                const __nv_bfloat162 hh = __floats2bfloat162_rn(pv[0], pv[1]);
                w[e2] = *reinterpret_cast<const uint32_t*>(&hh);
              }
              n_supp += (int)((cnt[0] + cnt[1]) + (cnt[2] + cnt[3]));
              s0 += (q0[0] + q0[1]) + (q0[2] + q0[3]);
              s1 += (q1[0] + q1[1]) + (q1[2] + q1[3]);
            } else {
#pragma unroll
              for (int e2 = 0; e2 < 16; ++e2) {
                float pv[2];
#pragma unroll
                for (int z = 0; z < 2; ++z) {
                  const int u = e2 * 2 + z;
                  const float yr = fmaf(ra, va[u], -tau);
                  const bool ok = valid && yr > 0.f && (!edge || col0 + u <= lim);
                  float ye1;
                  pow_pair_c<EC>(ok ? yr : 0.f, ok, a.expo, pv[z], ye1);
                  n_supp += ok ? 1 : 0;
                  s0 += pv[z];
                  s1 += ye1;
                }
                const __nv_bfloat162 hh = __floats2bfloat162_rn(pv[0], pv[1]);
                w[e2] = *reinterpret_cast<const uint32_t*>(&hh);
              }
            }
            // P of the previous tile must have been consumed before its buffer is rewritten
            alive = __all_sync(0xffffffffu, mbar_wait(p_empty, pphase ^ 1u, abort_flag));
            pphase ^= 1u;
            if (!alive) break;
            // shared memory, K-major with 128-byte swizzle: row r, 16-byte unit u of the 64-key block sits at
            // r*128 + ((u ^ (r & 7)) * 16)
            const uint32_t blk = p_smem + (uint32_t)(quarter >> 1) * (TM * 128) + (uint32_t)row_local * 128u;
#pragma unroll
            for (int u4 = 0; u4 < 4; ++u4) {
              const uint32_t unit = (uint32_t)((quarter & 1) * 4 + u4);
              const uint32_t addr = blk + ((unit ^ (uint32_t)(row_local & 7)) << 4);
              asm volatile("st.shared::cta.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w[4 * u4]),
                           "r"(w[4 * u4 + 1]), "r"(w[4 * u4 + 2]), "r"(w[4 * u4 + 3])
                           : "memory");
            }
            // make the P stores visible to the tensor core (async proxy), then hand the tile over
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full);
          }
        }
        if (!alive) break;
        // the next sweep's vote slot: its last readers (the roles deciding the kind of sweep s - 1, or the end of the
        // previous item) are past it once this sweep's tiles have come through
        if (warp == 2 && lane == 0) sts_u32(done_word + 4 * ((s + 1) % 3), 3u);
        if (output) {
          // all of this sweep's P V contractions have finished (its O stays in TMEM until the vote is in)
          alive = __all_sync(0xffffffffu, mbar_wait(o_full, ophase, abort_flag));
          ophase ^= 1u;
          if (!alive) break;
          n_supp_out = n_supp;
        }
        // ---- between sweeps: the threads of a row swap their partial results, Newton update, and the vote "every
        //      row of the tile has converged"
        {
          float r0[4], r1[4];
          alive = swap4(find_max ? ymax : s0, s1, r0, r1);
          if (!alive) break;
          if (find_max) {
            ymax = fmaxf(fmaxf(r0[0], r0[1]), fmaxf(r0[2], r0[3]));
          } else {
            s0 = (r0[0] + r0[1]) + (r0[2] + r0[3]);
            s1 = (r1[0] + r1[1]) + (r1[2] + r1[3]);
          }
        }
        const float mass_err = find_max ? 1.0f : fabsf((smp ? (float)kTileSampleStride * s0 : s0) - 1.0f);
        if (find_max) {
          it_tau = tau_iter_start(ymax);
          tau = it_tau.tau;
        } else if (!done) {
          if (smp) {
            // a sampled key stands for kTileSampleStride keys of the row: the sample is solved for that much mass, so
            // that its threshold estimates the row's instead of only bounding it from below
            s0 *= (float)kTileSampleStride;
            s1 *= (float)kTileSampleStride;
          }
          if (kind == kFullNewton && n_full == 1 && stiles > 0 && s0 < 0.999f && s1 > 0.f) {
            // the estimate was past the row's threshold: F = S^(1/e) - 1 is convex and decreasing, so one Newton step
            // from there lands at or before the root, and the iteration goes on from the left as usual
            it_tau.tau += threshold_step(s0, s1, a.expo_class, a.expo);
            tau = it_tau.tau;
          } else {
            // e >= 1: Newton from the left (e-norm step); e < 1: bracketed (see tau_iter_update)
            // (a looser stop -- a step of 1e-4 |tau| -- saves a sweep and keeps O and tau within tolerance, but the
            // backward pass, whose dQ is what survives the cancellation sum_j dS_ij = 0, needs the threshold to fp32)
            // (the sample's threshold is an estimate of the row's, a few per cent off in mass: no point in solving the
            // sample any finer than that)
            done = !tau_iter_update(it_tau, s0, s1, a.expo_class, a.expo, smp ? kSampleTol : 2e-6f);
            tau = it_tau.tau;
          }
          if (output && mass_err <= kOutputMass) done = true;
        }
        if (output && s >= kMaxSweeps - 1) done = true;   // the cap: this sweep's O is the result
        const bool near = done || mass_err <= kNearMass;
        const bool warp_done = __all_sync(0xffffffffu, done), warp_near = __all_sync(0xffffffffu, near);
        if (lane == 0) {
          const unsigned keep = find_max ? 0u : (warp_done ? 1u : 0u) | (warp_near ? 2u : 0u);
          if (keep != 3u) atomicAnd(reinterpret_cast<unsigned*>(__cvta_shared_to_generic(done_word + 4 * (s % 3))), keep);
          mbar_arrive(ctl);
        }
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (lds_u32(abort_flag)) {
    if (threadIdx.x == 0 && a.status) atomicOr(a.status + ENTMAX_ATTN_STATUS_FLAGS, ENTMAX_ATTN_FLAG_WAIT_EXPIRED);
    // the producer and the MMA issuer have waited for their copies and MMAs in flight; only if one of those waits ran
    // out as well is there nothing left but to give the hardware time
    if (lds_u32(drain_fail)) {
      const uint64_t t0 = global_ns();
      while (global_ns() - t0 < 200000ull) { }
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// Rewrites tile_list[0 .. *tile_count) in the order the dense-tile kernels hand the Q tiles out: on causal problems
// the tiles that see the most keys first (descending tile index, the heads interleaved).  The listed tiles are the
// ones flagged in tile_flag; the kernel compacts the flags in that order.  One CTA.
__global__ void __launch_bounds__(1024) order_tiles_kernel(const int32_t* __restrict__ tile_flag, int tiles_per_head,
                                                           int n_bh, int32_t* __restrict__ tile_list,
                                                           const int32_t* __restrict__ tile_count) {
  __shared__ int warp_sum[32];
  __shared__ int base;
  if (*tile_count == 0) return;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const long long total = (long long)tiles_per_head * n_bh;
  if (threadIdx.x == 0) base = 0;
  __syncthreads();
  for (long long c0 = 0; c0 < total; c0 += 1024) {
    const long long pos = c0 + threadIdx.x;
    int id = -1;
    bool f = false;
    if (pos < total) {
      const int tile = tiles_per_head - 1 - (int)(pos / n_bh);
      id = (int)(pos % n_bh) * tiles_per_head + tile;
      f = tile_flag[id] != 0;
    }
    const unsigned bal = __ballot_sync(0xffffffffu, f);
    if (lane == 0) warp_sum[w] = __popc(bal);
    __syncthreads();
    int off = base;
    for (int x = 0; x < w; ++x) off += warp_sum[x];
    if (f) tile_list[off + __popc(bal & ((1u << lane) - 1u))] = id;
    __syncthreads();
    if (threadIdx.x == 0) {
      int sum = 0;
      for (int x = 0; x < 32; ++x) sum += warp_sum[x];
      base += sum;
    }
    __syncthreads();
  }
}

template <int HD, int EC>
cudaError_t launch_tile_impl(const Problem& p, const void* q, const void* k, const void* v, const TileArgsK& args,
                             cudaStream_t stream) {
  CUtensorMap map_q, map_k, map_v;
  cudaError_t err = make_tile_map(&map_q, q, p.D, p.N, p.H, p.B, p.sn, p.sh, p.sb);
  if (err != cudaSuccess) return err;
  err = make_tile_map(&map_k, k, p.D, p.N, p.H, p.B, p.sn, p.sh, p.sb);
  if (err != cudaSuccess) return err;
  err = make_tile_map(&map_v, v, p.D, p.N, p.H, p.B, p.sn, p.sh, p.sb);
  if (err != cudaSuccess) return err;
  CUtensorMap map_ks = map_k;   // short sequences never take the sampled start
  if (p.N >= kSampleMinTiles * TN) {
    err = make_sampled_tile_map(&map_ks, k, p.D, p.N, p.H, p.B, p.sn, p.sh, p.sb, kTileSampleStride);
    if (err != cudaSuccess) return err;
  }
  err = cudaFuncSetAttribute(tile_fwd_kernel<HD, EC>, cudaFuncAttributeMaxDynamicSharedMemorySize, TCfg<HD>::kSmemBytes);
  if (err != cudaSuccess) return err;
  int dev = 0, sms = 0;
  err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;
  const long all_tiles = (long)p.B * p.H * args.tiles_per_head;
  const int grid = (int)(all_tiles < sms ? all_tiles : sms);
  tile_fwd_kernel<HD, EC><<<grid, kThreadsT, TCfg<HD>::kSmemBytes, stream>>>(map_q, map_k, map_v, map_ks, args);
  return cudaGetLastError();
}

}  // namespace

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

cudaError_t encode_fn(EncodeTiledFn* fn) {
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

}  // namespace

namespace sm100 {

// [B,H,N,D] bf16 tensor as a 4-D map (D, N, H, B); box = 64 columns (one 128-byte swizzle row) x box_rows rows
cudaError_t make_tile_map(CUtensorMap* map, const void* base, int D, int N, int H, int B, int64_t sn, int64_t sh,
                          int64_t sb, int box_rows) {
  EncodeTiledFn fn;
  cudaError_t err = encode_fn(&fn);
  if (err != cudaSuccess) return err;
  cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)N, (cuuint64_t)H, (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)sn * 2, (cuuint64_t)sh * 2, (cuuint64_t)sb * 2};
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t make_acc_map(CUtensorMap* map, const float* base, int D, int N, int BH) {
  EncodeTiledFn fn;
  cudaError_t err = encode_fn(&fn);
  if (err != cudaSuccess) return err;
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)N, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)D * 4, (cuuint64_t)N * D * 4};
  cuuint32_t box[3] = {32, 128, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t make_sampled_tile_map(CUtensorMap* map, const void* base, int D, int N, int H, int B, int64_t sn, int64_t sh,
                                  int64_t sb, int stride, int box_rows) {
  EncodeTiledFn fn;
  cudaError_t err = encode_fn(&fn);
  if (err != cudaSuccess) return err;
  const cuuint64_t groups = (cuuint64_t)(N / stride);
  cuuint64_t dims[5] = {(cuuint64_t)D, (cuuint64_t)stride, groups > 0 ? groups : 1, (cuuint64_t)H, (cuuint64_t)B};
  cuuint64_t strides[4] = {(cuuint64_t)sn * 2, (cuuint64_t)sn * 2 * stride, (cuuint64_t)sh * 2, (cuuint64_t)sb * 2};
  cuuint32_t box[5] = {64, 1, (cuuint32_t)box_rows, 1, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

}  // namespace sm100

cudaError_t order_tiles(const Problem& p, const int32_t* tile_flag, int32_t* tile_list, const int32_t* tile_count,
                        cudaStream_t stream) {
  if (!p.causal) return cudaSuccess;   // every Q tile sees the same keys: any order will do
  order_tiles_kernel<<<1, 1024, 0, stream>>>(tile_flag, (p.N + TM - 1) / TM, p.B * p.H, tile_list, tile_count);
  return cudaGetLastError();
}

cudaError_t launch_tile_fwd(const Problem& p, const void* q, const void* k, const void* v, const float* scale,
                            const int32_t* tile_flag, int32_t* tile_list, const int32_t* tile_count,
                            int32_t* work_counter, const int32_t* row_cnt, int32_t* dense_cnt, void* o, float* tau,
                            int32_t* status, cudaStream_t stream) {
  cudaError_t oerr = order_tiles(p, tile_flag, tile_list, tile_count, stream);
  if (oerr != cudaSuccess) return oerr;
  TileArgsK args;
  args.B = p.B; args.H = p.H; args.N = p.N;
  args.causal = p.causal;
  args.expo_class = p.expo_class;
  args.expo = p.expo;
  args.alpha_m1 = p.alpha - 1.0f;
  args.sm_scale = p.sm_scale;
  args.scale = scale;
  args.alibi = p.alibi;
  args.scale_sb = p.scale_sb;
  args.tile_list = tile_list;
  args.tile_count = tile_count;
  args.work_counter = work_counter;
  args.row_cnt = row_cnt;
  args.dense_cnt = dense_cnt;
  args.o = o;
  args.tau = tau;
  args.sb = p.sb; args.sh = p.sh; args.sn = p.sn;
  args.status = status;
  args.tiles_per_head = (p.N + TM - 1) / TM;
#define ENTMAX_TILE_FWD(EC)                                                  \
  (p.D == 64 ? launch_tile_impl<64, EC>(p, q, k, v, args, stream)             \
             : launch_tile_impl<128, EC>(p, q, k, v, args, stream))
  switch (p.expo_class) {
    case kExpo2: return ENTMAX_TILE_FWD(kExpo2);
    case kExpo1: return ENTMAX_TILE_FWD(kExpo1);
    case kExpo4: return ENTMAX_TILE_FWD(kExpo4);
    default: return ENTMAX_TILE_FWD(kExpoGeneral);
  }
#undef ENTMAX_TILE_FWD
}

}  // namespace entmax
