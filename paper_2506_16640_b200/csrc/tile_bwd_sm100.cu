// Dense-tile backward for bf16 problems on sm_100a: the rows whose support does not fit the sparse
// lists are differentiated tile by tile on the tensor cores.  With y_ij = (alpha-1) c_i z_ij - tau_i,
// p_ij = [y_ij]_+^e (Eq. 1) and u_ij = [y_ij]_+^(e-1) = p_ij^(2-alpha), the entmax Jacobian gives
//   dP_ij = dO_i . v_j,   rho_i = sum_j u_ij dP_ij / sum_j u_ij,   dS_ij = u_ij (dP_ij - rho_i),
//   dQ_i = g_i sum_j dS_ij k_j,   dK_j = sum_i g_i dS_ij q_i,   dV_j = sum_i p_ij dO_i,
//   dL/dc_i = sum_j dS_ij z_ij                      (g_i = c_i * sm_scale, c_i the ASEntmax scale)
// Two kernels.  tile_bwd_kernel, query-major: a work item is one Q tile of 128 rows that holds at least one such
// row; two passes over its visible K/V tiles:
//   pass A   S = Q K^T and dP = dO V^T into TMEM; the row threads accumulate sum u and sum u dP: rho_i (kept for the
//            second kernel);
//   pass B   S and dP again; the row threads write g dS (bf16, and what the rounding left over) to shared memory;
//            dQ += (g dS) K     (A = g dS K-major, B = K tile with the head dim contiguous)   kept in TMEM.
// tile_bwd_kv_kernel, key-major: a work item is one K/V tile; over the marked Q tiles that see it, S and dP once
// more, P and g dS to shared memory, and
//            dK_t += (g dS)^T Q (A = the shared tile read M-major, B = Q tile, head dim contiguous)
//            dV_t += P^T dO     (likewise), accumulated in TMEM over those Q tiles and added to the fp32 dK / dV
//            accumulators in global memory once per K/V tile, by bulk tensor reductions from a staging tile.
// (One kernel that also formed dK_t and dV_t per (Q tile, K tile) pair was bound by those reductions in L2: 128 KB of
// them per pair.)  Rows of a Q tile that are not marked contribute zeros (their P and dS rows are written as zero)
// and their dQ is not stored: the list kernels have already handled them.
//
// CTA: warp 0 TMA producer, warp 1 MMA issuer, warps 2..17 four threads per TMEM lane (32 columns each).  Every wait is
// bounded (see sm100_ptx.cuh); on expiry the CTA flags the call's status word and leaves.
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace entmax {

namespace {

using namespace sm100;

constexpr int TM = 128;            // query rows per item = TMEM lanes
constexpr int TN = 128;            // keys per K/V tile
constexpr int kConsGroups = 4;                       // threads per TMEM lane
constexpr int kConsWarps = 4 * kConsGroups;           // four lane quadrants each
constexpr int kThreadsB = (2 + kConsWarps) * 32;      // TMA warp, MMA warp, the consumer warps
constexpr int kTileBytes = TM * TN * 2;   // P or dS tile, bf16

template <int HD>
struct BCfg {
  static constexpr int kHalves = HD / 64;
  static constexpr int kQBytes = TM * HD * 2;       // Q tile; also dO, K, V tiles
  static constexpr int kBarBytes = 256;
  static constexpr int kSmemBytes = 4 * kQBytes + 3 * kTileBytes + 1024 + kBarBytes;
  static_assert(kSmemBytes <= 232448, "shared memory of one CTA");
  static constexpr int kTmemS = 0, kTmemDP = TN, kTmemDQ = 2 * TN;
};

struct TileBwdArgs {
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
  const uint32_t* tile_mask; // [tiles, 4]: bit r of a tile's 128-bit mask marks row r for this kernel
  const float* tau;
  void* dq;                  // bf16 [B,H,N,D]
  float* acc_dk;             // fp32 [B,H,N,D] contiguous
  float* acc_dv;
  float* dc_rows;            // [B,H,N] or nullptr
  float* rho;                // [B,H,N]: rho_i of the marked rows, from the query-major to the key-major kernel
  const int32_t* tile_flag;  // [tiles]: nonzero for the Q tiles in tile_list
  int32_t* kv_counter;       // next item of the key-major kernel (zero on entry)
  int64_t sb, sh, sn;
  int32_t* status;
  int tiles_per_head;
};

// A, B bf16 K-major, fp32 accumulate, M = 128, N = TN (S = Q K^T and dP = dO V^T)
__host__ __device__ constexpr uint32_t idesc_kk() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TN >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
}
// A K-major, B with N contiguous (bit 16), N = HD (dQ += dS K)
template <int HD>
__host__ __device__ constexpr uint32_t idesc_kn() {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(HD >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
}
// A with M contiguous (bit 15), B with N contiguous (bit 16), N = HD (dK = dS^T Q, dV = P^T dO)
template <int HD>
__host__ __device__ constexpr uint32_t idesc_mn() {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(HD >> 3) << 17) |
         ((uint32_t)(TM >> 4) << 24);
}
// Low descriptor word of a [128 x 64-element-blocks] tile read with its 128-byte rows as the M (or N)
// direction, 128-byte swizzle: a swizzle atom is one 128-byte row of 64 elements by 8 rows; atoms repeat
// every 1024 bytes along the rows (stride-dimension offset, in the high word) and every 128*128 bytes from
// one 64-element block to the next (leading-dimension offset).  Sixteen rows (one MMA K step) are 2048 bytes.
__device__ __forceinline__ uint32_t mn_desc_lo(uint32_t saddr) {
  return ((saddr & 0x3FFFFu) >> 4) | ((uint32_t)((128 * 128) >> 4) << 16);
}

// m^(e-1) of a clamped m >= 0 for the compile-time exponent classes (0 for m = 0, also for e = 1), FMA-pipe work only
template <int EC>
__device__ __forceinline__ float clamped_pow_m1(float m) {
  if constexpr (EC == kExpo2) return m;
  else if constexpr (EC == kExpo4) return (m * m) * m;
  else return positive_indicator(m);
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  const __nv_bfloat162 hh = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&hh);
}

// Marks the rows of row_list[0 .. *row_count) in the per-tile masks and lists every tile once.
__global__ void mark_tiles_kernel(int N, int tiles_per_head, const int32_t* __restrict__ row_list,
                                  const int32_t* __restrict__ row_count, uint32_t* __restrict__ tile_mask,
                                  int32_t* __restrict__ tile_flag, int32_t* __restrict__ tile_list,
                                  int32_t* __restrict__ tile_count) {
  const int total = *row_count;
  for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < total; t += gridDim.x * blockDim.x) {
    const int grow = row_list[t];
    const int bh = grow / N, i = grow - bh * N;
    const int id = bh * tiles_per_head + i / TM;
    const int r = i % TM;
    atomicOr(tile_mask + 4 * (size_t)id + (r >> 5), 1u << (r & 31));
    if (atomicExch(tile_flag + id, 1) == 0) tile_list[atomicAdd(tile_count, 1)] = id;
  }
}

template <int HD, int EC>
__global__ void __launch_bounds__(kThreadsB, 1) tile_bwd_kernel(const __grid_constant__ CUtensorMap map_q,
                                                               const __grid_constant__ CUtensorMap map_k,
                                                               const __grid_constant__ CUtensorMap map_v,
                                                               const __grid_constant__ CUtensorMap map_do,
                                                               const TileBwdArgs a) {
  using C = BCfg<HD>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_smem = sbase;
  const uint32_t do_smem = q_smem + C::kQBytes;
  const uint32_t k_smem = do_smem + C::kQBytes;
  const uint32_t v_smem = k_smem + C::kQBytes;
  const uint32_t p_smem = v_smem + C::kQBytes;           // (the key-major kernel's P tile; here: second K stage)
  const uint32_t ds_smem = p_smem + kTileBytes;           // g dS tile (bf16), same layout
  const uint32_t dl_smem = ds_smem + kTileBytes;          // what the bf16 rounding of g dS left over, same layout
  const uint32_t bars = dl_smem + kTileBytes;
  const uint32_t qdo_full = bars, qdo_empty = bars + 8;
  const uint32_t k_full0 = bars + 16, k_empty0 = bars + 24;
  const uint32_t sd_full = bars + 32, sd_empty = bars + 40;
  const uint32_t pds_full = bars + 48, pds_empty = bars + 56;
  const uint32_t dq_full = bars + 80, dq_empty = bars + 88;
  const uint32_t tmem_slot = bars + 96;
  const uint32_t abort_flag = bars + 100;
  const uint32_t drain_bar = bars + 104;      // teardown: every MMA issued so far has finished
  const uint32_t drain_fail = bars + 112;     // uint32: a teardown wait ran out as well
  const uint32_t w_full = bars + 120;         // [2] a work item has been published
  const uint32_t w_empty = bars + 136;        // [2] ... and read by the MMA issuer and every consumer warp
  const uint32_t w_item = bars + 152;         // int32 [2]: tile id, -1 = no more work
  const uint32_t x_bar = bars + 160;          // the threads of a row have written their partial sums
  const uint32_t v_full0 = bars + 168, v_empty0 = bars + 176;
  // Pass A has a second K / V stage: the P tile's buffer (the key-major kernel's; idle here) and the g dS buffer, which
  // is idle until pass B and free again when the item's last contraction has finished -- which the producer waits for
  // before it loads anything of the next item.
  const uint32_t k_full1 = bars + 184, k_empty1 = bars + 192, v_full1 = bars + 200, v_empty1 = bars + 208;
  auto k_full = [&](int st) { return st ? k_full1 : k_full0; };
  auto k_empty = [&](int st) { return st ? k_empty1 : k_empty0; };
  auto v_full = [&](int st) { return st ? v_full1 : v_full0; };
  auto v_empty = [&](int st) { return st ? v_empty1 : v_empty0; };
  auto k_stage = [&](int st) { return st ? p_smem : k_smem; };
  auto v_stage = [&](int st) { return st ? ds_smem : v_smem; };

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int n_tiles = *a.tile_count;

  if (threadIdx.x == 0) {
    mbar_init(qdo_full, 1);
    mbar_init(qdo_empty, 1);
    for (int st = 0; st < 2; ++st) {
      mbar_init(k_full(st), 1);
      mbar_init(k_empty(st), 1);
      mbar_init(v_full(st), 1);
      mbar_init(v_empty(st), 1);
    }
    mbar_init(sd_full, 1);
    mbar_init(sd_empty, kConsWarps);
    mbar_init(pds_full, kConsWarps);
    mbar_init(pds_empty, 1);
    mbar_init(dq_full, 1);
    mbar_init(dq_empty, kConsWarps);
    mbar_init(x_bar, kConsWarps);
    mbar_init(drain_bar, 1);
    for (int t = 0; t < 2; ++t) {
      mbar_init(w_full + 8 * t, 1);
      mbar_init(w_empty + 8 * t, 1 + kConsWarps);   // MMA issuer + the consumer warps
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

  auto item_tiles = [&](int tile) -> int {
    const int row0 = tile * TM;
    if (!a.causal) return (a.N + TN - 1) / TN;
    int last_row = row0 + TM - 1;
    if (last_row > a.N - 1) last_row = a.N - 1;
    return last_row / TN + 1;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    // (the whole warp runs the control flow, one elected lane issues the copies: see the MMA issuer).  K and V
    // tiles have barriers of their own: in pass B the V tile is free again once dP has been formed and the K tile
    // once dQ has taken it, so the next tile's copies run under the dK / dV contractions of this one.
    {
      uint32_t kbits = 0, vbits = 0 /* bit st: times the stage's barrier has been armed, mod 2 */, qphase = 0, wphase = 0;
      int slot = 0;
      bool alive = true;
      auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
      };
      while (alive) {
        // items are handed out from a shared counter, in the list's order (longest first on causal problems)
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
        const int tiles = item_tiles(tile);
        alive = wait_all(qdo_empty, qphase ^ 1u);
        if (!alive) break;
        qphase ^= 1u;
        if (elect_one()) {
          mbar_expect_tx(qdo_full, 2 * C::kQBytes);
          for (int hf = 0; hf < C::kHalves; ++hf) {
            tma_load_4d(q_smem + hf * (TM * 128), &map_q, qdo_full, hf * 64, tile * TM, h, b);
            tma_load_4d(do_smem + hf * (TM * 128), &map_do, qdo_full, hf * 64, tile * TM, h, b);
          }
        }
        __syncwarp();
        for (int t = 0; t < 2 * tiles && alive; ++t) {
          const int kt = t < tiles ? t : t - tiles;
          // K alternates between its two stages in both passes (the second one is a tile this kernel has no other use
          // for); V does so in pass A only: its second stage is the dS tile of pass B, where a V tile is free again as
          // soon as dP has been formed
          const int st = t < tiles ? (t & 1) : 0, kst = t & 1;
          alive = wait_all(v_empty(st), ((vbits >> st) & 1u) ^ 1u);
          if (!alive) break;
          vbits ^= 1u << st;
          if (elect_one()) {
            mbar_expect_tx(v_full(st), C::kQBytes);
            for (int hf = 0; hf < C::kHalves; ++hf)
              tma_load_4d(v_stage(st) + hf * (TN * 128), &map_v, v_full(st), hf * 64, kt * TN, h, b);
          }
          __syncwarp();
          alive = wait_all(k_empty(kst), ((kbits >> kst) & 1u) ^ 1u);
          if (!alive) break;
          kbits ^= 1u << kst;
          if (elect_one()) {
            mbar_expect_tx(k_full(kst), C::kQBytes);
            for (int hf = 0; hf < C::kHalves; ++hf)
              tma_load_4d(k_stage(kst) + hf * (TN * 128), &map_k, k_full(kst), hf * 64, kt * TN, h, b);
          }
          __syncwarp();
        }
      }
      if (!alive && lane == 0) {
        // a wait ran out somewhere in the CTA: the copies this warp armed barriers for must land before shared
        // memory goes away (after n arms a phase word holds n mod 2 and the last armed phase has the other parity)
        bool ok = mbar_drain(qdo_full, qphase ^ 1u);
        for (int st = 0; st < 2; ++st) {
          ok &= mbar_drain(k_full(st), ((kbits >> st) & 1u) ^ 1u);
          ok &= mbar_drain(v_full(st), ((vbits >> st) & 1u) ^ 1u);
        }
        if (!ok) sts_u32(drain_fail, 1u);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp runs the control flow (waits are voted on, what is read from shared memory is broadcast), so
    // that descriptors, addresses and counters are warp-uniform; one elected lane issues the tensor-core
    // instructions.
    {
      constexpr uint32_t id_kk = idesc_kk();
      constexpr uint32_t id_kn = idesc_kn<HD>();
      const uint64_t hi = (uint64_t)kDescHi << 32;
      const uint64_t q_d = hi | smem_desc_lo(q_smem), do_d = hi | smem_desc_lo(do_smem);
      const uint64_t k_d = hi | smem_desc_lo(k_smem), v_d = hi | smem_desc_lo(v_smem);
      const uint64_t ds_d = hi | smem_desc_lo(ds_smem), dl_d = hi | smem_desc_lo(dl_smem);
      const uint64_t k_n_d = hi | mn_desc_lo(k_smem), k1_n_d = hi | mn_desc_lo(p_smem);
      uint32_t kbits = 0, vbits = 0 /* bit st: phase of the stage's barrier to wait for */, qphase = 0, sdphase = 0,
               pdsphase = 0, dqphase = 0, wphase = 0;
      const uint64_t k1_d = hi | smem_desc_lo(p_smem), v1_d = hi | smem_desc_lo(ds_smem);   // stage 1 of pass A
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
        const int tiles = item_tiles(tile);
        alive = wait_all(qdo_full, qphase);
        qphase ^= 1u;
        if (!alive) break;
        // S = Q K^T and dP = dO V^T of tile t (pass A: t < tiles, pass B: the same tiles again)
        auto issue_sd = [&](int t) -> bool {
          const bool pass_b = t >= tiles;
          const int st = pass_b ? 0 : (t & 1), kst = t & 1;
          bool ok = wait_all(k_full(kst), (kbits >> kst) & 1u);
          kbits ^= 1u << kst;
          if (ok) ok = wait_all(v_full(st), (vbits >> st) & 1u);
          vbits ^= 1u << st;
          const uint64_t ks_d = kst ? k1_d : k_d, vs_d = st ? v1_d : v_d;
          if (ok) ok = wait_all(sd_empty, sdphase ^ 1u);
          if (!ok) return false;
          sdphase ^= 1u;
          tc_fence_after();
          if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < HD / 16; ++kk) {
              const uint32_t off = (kk >> 2) * ((TM * 128) >> 4) + (kk & 3) * 2;
              umma_bf16_desc(tmem_base + C::kTmemS, q_d + off, ks_d + off, id_kk, kk > 0 ? 1u : 0u);
            }
#pragma unroll
            for (int kk = 0; kk < HD / 16; ++kk) {
              const uint32_t off = (kk >> 2) * ((TM * 128) >> 4) + (kk & 3) * 2;
              umma_bf16_desc(tmem_base + C::kTmemDP, do_d + off, vs_d + off, id_kk, kk > 0 ? 1u : 0u);
            }
            umma_commit(sd_full);
            umma_commit(v_empty(st));          // dP has been formed: the V tile is free
            if (!pass_b) umma_commit(k_empty(kst));
          }
          __syncwarp();
          return true;
        };
        for (int t = 0; t < tiles && alive; ++t) alive = issue_sd(t);
        if (alive) {
          // the previous item's dQ must have been read before this item's first dQ MMA overwrites it
          alive = wait_all(dq_empty, dqphase ^ 1u);
          dqphase ^= 1u;
        }
        if (alive) alive = issue_sd(tiles);
        for (int t = tiles; t < 2 * tiles && alive; ++t) {
          // the next tile's S and dP are issued before this tile's dS is waited for (its K tile sits in the other
          // stage), so that they run while the consumers form dS
          if (t + 1 < 2 * tiles) {
            alive = issue_sd(t + 1);
            if (!alive) break;
          }
          const int kst = t & 1;
          const uint64_t kn_d = kst ? k1_n_d : k_n_d;
          // g dS of this tile and its rounding remainder are in shared memory
          alive = wait_all(pds_full, pdsphase);
          pdsphase ^= 1u;
          if (!alive) break;
          tc_fence_after();
          if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < TN / 16; ++kk) {
              const uint32_t a_off = (kk >> 2) * ((TM * 128) >> 4) + (kk & 3) * 2;   // 64 keys per 128-byte row
              const uint32_t b_off = kk * ((16 * 128) >> 4);                           // 16 keys = 16 rows of 128 B
              umma_bf16_desc(tmem_base + C::kTmemDQ, ds_d + a_off, kn_d + b_off, id_kn, (t > tiles || kk > 0) ? 1u : 0u);
            }
            // the rounding remainder of g dS as a second operand: the rows of dS sum to zero, so when a row's keys
            // are nearly equal vectors (retrieval: several copies of one key) dQ is what is left after a
            // cancellation, and the bf16 rounding of dS alone (2^-9 of every term) would be a large part of it
#pragma unroll
            for (int kk = 0; kk < TN / 16; ++kk) {
              const uint32_t a_off = (kk >> 2) * ((TM * 128) >> 4) + (kk & 3) * 2;
              const uint32_t b_off = kk * ((16 * 128) >> 4);
              umma_bf16_desc(tmem_base + C::kTmemDQ, dl_d + a_off, kn_d + b_off, id_kn, 1u);
            }
            umma_commit(k_empty(kst));         // dQ has taken the K tile
            umma_commit(pds_empty);
            if (t == 2 * tiles - 1) umma_commit(dq_full);
          }
          __syncwarp();
        }
        if (elect_one()) umma_commit(qdo_empty);
        __syncwarp();
      }
      if (!alive && lane == 0) {
        // the tensor core must be done with shared memory and TMEM before they are released
        umma_commit(drain_bar);
        if (!mbar_drain(drain_bar, 0u)) sts_u32(drain_fail, 1u);
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers: four threads per TMEM lane
    // (warps w, w + 4, w + 8, w + 12 share a lane quadrant; `quarter` picks the 32 of a tile's 128 columns -- or
    // the 32-column chunk of a head-dim-wide accumulator -- a thread works on)
    const int quad = warp & 3;
    const int quarter = (warp - 2) >> 2;
    const int row_local = quad * 32 + lane;
    const uint32_t taddr_row = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint32_t sdphase = 0, pdsphase = 0, dqphase = 0, wphase = 0, xphase = 0;
    int slot = 0;
    bool alive = true;
    // The four threads of a row swap partial sums through shared memory.  The slots live in the remainder tile's
    // buffer, which is idle whenever a swap happens (between the passes: not yet written; after the item's last
    // contraction: no longer read); a second round of the barrier keeps a fast warp from rewriting the buffer while
    // a slow one still reads it.  All four threads add the same four numbers in the same order.
    auto swap4 = [&](float x0, float x1, float& r0, float& r1) -> bool {
      const uint32_t mine = dl_smem + (uint32_t)(quarter * TM + row_local) * 8u;
      sts_u32(mine, __float_as_uint(x0));
      sts_u32(mine + 4, __float_as_uint(x1));
      __syncwarp();
      if (lane == 0) mbar_arrive(x_bar);
      bool ok = __all_sync(0xffffffffu, mbar_wait(x_bar, xphase, abort_flag));
      xphase ^= 1u;
      if (!ok) return false;
      float a0[kConsGroups], a1[kConsGroups];
#pragma unroll
      for (int gq = 0; gq < kConsGroups; ++gq) {
        a0[gq] = __uint_as_float(lds_u32(dl_smem + (uint32_t)(gq * TM + row_local) * 8u));
        a1[gq] = __uint_as_float(lds_u32(dl_smem + (uint32_t)(gq * TM + row_local) * 8u + 4u));
      }
      r0 = (a0[0] + a0[1]) + (a0[2] + a0[3]);
      r1 = (a1[0] + a1[1]) + (a1[2] + a1[3]);
      __syncwarp();
      if (lane == 0) mbar_arrive(x_bar);
      ok = __all_sync(0xffffffffu, mbar_wait(x_bar, xphase, abort_flag));
      xphase ^= 1u;
      return ok;
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
      const int tiles = item_tiles(tile);
      const int i = tile * TM + row_local;
      const bool valid = i < a.N;
      const bool marked = valid && ((a.tile_mask[4 * (size_t)id + (row_local >> 5)] >> (row_local & 31)) & 1u);
      const size_t grow = (size_t)bh * a.N + (valid ? i : 0);
      const int lim = a.causal ? i : a.N - 1;
      const float c_i = valid ? a.scale[(size_t)b * a.scale_sb + (size_t)h * a.N + i] : 0.f;
      const float ra = a.alpha_m1 * (c_i * a.sm_scale);
      const float g = c_i * a.sm_scale;
      const float slope = a.alibi ? a.alibi[h] / a.sm_scale : 0.f;   // bias in accumulator units
      const float tau = marked ? a.tau[grow] : 0.f;
      const float ra_m = marked ? ra : 0.f;
      float su = 0.f, sud = 0.f, rho = 0.f;
      float dcs[2] = {0.f, 0.f};   // sum_j dS_ij * (accumulator + bias), two partial sums
      for (int t = 0; t < 2 * tiles && alive; ++t) {
        const bool pass_b = t >= tiles;
        const int kt = pass_b ? t - tiles : t;
        if (t == tiles) {
          // rho of the row from the four threads' shares of sum u and sum u dP
          float su_all, sud_all;
          alive = swap4(su, sud, su_all, sud_all);
          if (!alive) break;
          rho = su_all > 0.f ? sud_all / su_all : 0.f;
          if (marked && quarter == 0) a.rho[grow] = rho;   // for the key-major kernel
        }
        alive = __all_sync(0xffffffffu, mbar_wait(sd_full, sdphase, abort_flag));
        if (!alive) break;
        sdphase ^= 1u;
        tc_fence_after();
        // this thread's 32 columns, 16 at a time
#pragma unroll 1
        for (int hc = 0; hc < 2; ++hc) {
          float sa[16], dp[16];
          tmem_ld16(taddr_row + C::kTmemS + quarter * 32 + hc * 16, sa);
          tmem_ld16(taddr_row + C::kTmemDP + quarter * 32 + hc * 16, dp);
          tmem_ld_wait();
          const int col0 = kt * TN + quarter * 32 + hc * 16;
          if (slope != 0.f) {
#pragma unroll
            for (int u = 0; u < 16; ++u) sa[u] = fmaf(slope, (float)(col0 + u - i), sa[u]);
          }
          const bool edge = col0 + 15 > lim;
          if (!pass_b) {
            // four independent partial sums each, so that the additions do not form one serial chain
            float p0[4] = {0.f, 0.f, 0.f, 0.f}, p1[4] = {0.f, 0.f, 0.f, 0.f};
            if (EC != kExpoGeneral && !edge) {
              // away from the mask: one ALU-pipe clamp per element, the rest FMA-pipe work
#pragma unroll
              for (int u = 0; u < 16; ++u) {
                const float m = fmaxf(fmaf(ra, sa[u], -tau), 0.f);
                const float ye1 = clamped_pow_m1<EC>(m);
                p0[u & 3] += ye1;
                p1[u & 3] = fmaf(ye1, dp[u], p1[u & 3]);
              }
            } else {
#pragma unroll
              for (int u = 0; u < 16; ++u) {
                const float yr = fmaf(ra, sa[u], -tau);
                const bool ok = yr > 0.f && (!edge || col0 + u <= lim);
                float ye, ye1;
                pow_pair_c<EC>(ok ? yr : 0.f, ok, a.expo, ye, ye1);
                p0[u & 3] += ye1;
                p1[u & 3] = fmaf(ye1, dp[u], p1[u & 3]);
              }
            }
            su += (p0[0] + p0[1]) + (p0[2] + p0[3]);
            sud += (p1[0] + p1[1]) + (p1[2] + p1[3]);
          } else {
            // P and g dS -> bf16 -> shared memory, K-major with 128-byte swizzle: row r, 16-byte unit u of
            // the 64-key block sits at r*128 + ((u ^ (r & 7)) * 16)
            const uint32_t blk = (uint32_t)(quarter >> 1) * (TM * 128) + (uint32_t)row_local * 128u;
#pragma unroll
            for (int u4 = 0; u4 < 2; ++u4) {
              float dv[8], dl[8];
              if (EC != kExpoGeneral && !edge) {
                // away from the mask (an unmarked row has a = 0, tau = 0 here: every entry clamps to zero)
#pragma unroll
                for (int z = 0; z < 8; ++z) {
                  const int u = u4 * 8 + z;
                  const float m = fmaxf(fmaf(ra_m, sa[u], -tau), 0.f);
                  const float ds = clamped_pow_m1<EC>(m) * (dp[u] - rho);
                  dv[z] = g * ds;
                  dcs[z & 1] = fmaf(ds, sa[u], dcs[z & 1]);
                }
              } else {
#pragma unroll
                for (int z = 0; z < 8; ++z) {
                  const int u = u4 * 8 + z;
                  const float yr = fmaf(ra, sa[u], -tau);
                  const bool ok = marked && yr > 0.f && (!edge || col0 + u <= lim);
                  float ye, ye1;
                  pow_pair_c<EC>(ok ? yr : 0.f, ok, a.expo, ye, ye1);
                  const float ds = ye1 * (dp[u] - rho);
                  dv[z] = g * ds;
                  dcs[z & 1] = fmaf(ds, sa[u], dcs[z & 1]);
                }
              }
              // what the bf16 rounding of g dS leaves over, two entries at a time
#pragma unroll
              for (int z = 0; z < 8; z += 2) {
                const float2 r2 = __bfloat1622float2(__floats2bfloat162_rn(dv[z], dv[z + 1]));
                dl[z] = dv[z] - r2.x;
                dl[z + 1] = dv[z + 1] - r2.y;
              }
              if (hc == 0 && u4 == 0) {
                // g dS of the previous tile and its remainder must have been consumed before their buffers are
                // rewritten (waited for here, not before the loads: that tile's dQ contraction runs under this
                // tile's first element code)
                alive = __all_sync(0xffffffffu, mbar_wait(pds_empty, pdsphase ^ 1u, abort_flag));
                pdsphase ^= 1u;
              }
              if (!alive) continue;
              const uint32_t unit = (uint32_t)((quarter & 1) * 4 + hc * 2 + u4);
              const uint32_t off = blk + ((unit ^ (uint32_t)(row_local & 7)) << 4);
              asm volatile("st.shared::cta.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(ds_smem + off),
                           "r"(pack_bf16(dv[0], dv[1])), "r"(pack_bf16(dv[2], dv[3])), "r"(pack_bf16(dv[4], dv[5])),
                           "r"(pack_bf16(dv[6], dv[7]))
                           : "memory");
              asm volatile("st.shared::cta.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dl_smem + off),
                           "r"(pack_bf16(dl[0], dl[1])), "r"(pack_bf16(dl[2], dl[3])), "r"(pack_bf16(dl[4], dl[5])),
                           "r"(pack_bf16(dl[6], dl[7]))
                           : "memory");
            }
          }
        }
        if (!alive) break;
        // S and dP have been read
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(sd_empty);
        if (!pass_b) continue;
        // make the P / dS stores visible to the tensor core (async proxy), then hand the tiles over
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(pds_full);
      }
      if (!alive) break;
      // ---- dQ of the item
      alive = __all_sync(0xffffffffu, mbar_wait(dq_full, dqphase, abort_flag));
      dqphase ^= 1u;
      if (!alive) break;
      tc_fence_after();
      __nv_bfloat16* dqrow =
          reinterpret_cast<__nv_bfloat16*>(a.dq) + (size_t)b * a.sb + (size_t)h * a.sh + (size_t)i * a.sn;
      for (int c = quarter; c < HD / 32; c += kConsGroups) {
        float va[32];
        tmem_ld32(taddr_row + C::kTmemDQ + c * 32, va);
        tmem_ld_wait();
        if (marked) {
#pragma unroll
          for (int u8 = 0; u8 < 4; ++u8)
            *reinterpret_cast<uint4*>(dqrow + c * 32 + u8 * 8) =
                make_uint4(pack_bf16(va[u8 * 8], va[u8 * 8 + 1]), pack_bf16(va[u8 * 8 + 2], va[u8 * 8 + 3]),
                           pack_bf16(va[u8 * 8 + 4], va[u8 * 8 + 5]), pack_bf16(va[u8 * 8 + 6], va[u8 * 8 + 7]));
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(dq_empty);
      // dL/dc_i = sum_j dS_ij z_ij with z_ij = sm_scale * (accumulator + bias in accumulator units); every
      // contraction of the item has finished (dq_full), so the swap buffer is free
      if (a.dc_rows) {
        float dc_all, unused;
        alive = swap4(dcs[0] + dcs[1], 0.f, dc_all, unused);
        if (!alive) break;
        if (marked && quarter == 0) a.dc_rows[grow] = dc_all * a.sm_scale;
      }
      if (a.status && threadIdx.x == 64) atomicAdd(a.status + ENTMAX_ATTN_STATUS_TILES, 1);
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

// Key-major pass of the dense-tile backward: dK and dV of the marked Q tiles.  A work item is one K/V tile (128 keys
// of one head); it walks the head's marked Q tiles that see it, recomputes S = Q K^T and dP = dO V^T, forms P and
// g dS with the thresholds and the rho the query-major pass left in global memory, and accumulates
//   dK_t += (g dS)^T Q   and   dV_t += P^T dO
// in TMEM over all those Q tiles, so that each K/V tile is added to the fp32 accumulators once (by bulk tensor
// reductions from a staging tile) instead of once per (Q tile, K tile) pair -- the reductions in L2 were what bounded
// the single-kernel form.  Same roles and conventions as tile_bwd_kernel.
template <int HD, int EC>
__global__ void __launch_bounds__(kThreadsB, 1) tile_bwd_kv_kernel(const __grid_constant__ CUtensorMap map_q,
                                                                  const __grid_constant__ CUtensorMap map_k,
                                                                  const __grid_constant__ CUtensorMap map_v,
                                                                  const __grid_constant__ CUtensorMap map_do,
                                                                  const __grid_constant__ CUtensorMap map_dk,
                                                                  const __grid_constant__ CUtensorMap map_dv,
                                                                  const TileBwdArgs a) {
  using C = BCfg<HD>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_smem = sbase;
  const uint32_t do_smem = q_smem + C::kQBytes;
  const uint32_t k_smem = do_smem + C::kQBytes;
  const uint32_t v_smem = k_smem + C::kQBytes;
  const uint32_t p_smem = v_smem + C::kQBytes;           // P tile, [128 rows][128 keys] bf16, swizzled
  const uint32_t ds_smem = p_smem + kTileBytes;           // g dS tile (bf16), same layout; with P the staging tile
  const uint32_t bars = ds_smem + 2 * kTileBytes;         // (the query-major kernel's layout: the third tile is unused)
  const uint32_t qdo_full = bars, qdo_empty = bars + 8;
  const uint32_t kv_full = bars + 16, kv_empty = bars + 24;
  const uint32_t sd_full = bars + 32, sd_empty = bars + 40;
  const uint32_t pds_full = bars + 48, pds_empty = bars + 56;
  const uint32_t acc_full = bars + 64, acc_empty = bars + 72;
  const uint32_t tmem_slot = bars + 96;
  const uint32_t abort_flag = bars + 100;
  const uint32_t drain_bar = bars + 104;
  const uint32_t drain_fail = bars + 112;
  const uint32_t w_full = bars + 120;         // [2]
  const uint32_t w_empty = bars + 136;        // [2]
  const uint32_t w_item = bars + 152;         // int32 [2]: item, -1 = no more work
  const uint32_t x_bar = bars + 160;
  constexpr int kTmemDK = 2 * TN, kTmemDV = 2 * TN + 128;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int n_bh = a.B * a.H;
  const int n_items = (*a.tile_count > 0) ? n_bh * a.tiles_per_head : 0;   // nothing marked: nothing to do

  if (threadIdx.x == 0) {
    mbar_init(qdo_full, 1);
    mbar_init(qdo_empty, 1);
    mbar_init(kv_full, 1);
    mbar_init(kv_empty, 1);
    mbar_init(sd_full, 1);
    mbar_init(sd_empty, kConsWarps);
    mbar_init(pds_full, kConsWarps);
    mbar_init(pds_empty, 1);
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, kConsWarps);
    mbar_init(x_bar, kConsWarps);
    mbar_init(drain_bar, 1);
    for (int t = 0; t < 2; ++t) {
      mbar_init(w_full + 8 * t, 1);
      mbar_init(w_empty + 8 * t, 1 + kConsWarps);
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

  // Items are numbered kt * n_bh + bh: on causal problems the K tiles most Q tiles see come first.  The Q tiles of an
  // item: the head's marked ones, from the tile that holds the K tile's own rows on (causal) or all of them.
  auto first_q = [&](int kt) -> int { return a.causal ? kt : 0; };
  auto next_marked = [&](int bh, int qt) -> int {      // first marked Q tile >= qt of head bh, or tiles_per_head
    while (qt < a.tiles_per_head && a.tile_flag[bh * a.tiles_per_head + qt] == 0) ++qt;
    return qt;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    uint32_t kvphase = 0, qphase = 0, wphase = 0;
    int slot = 0;
    bool alive = true;
    auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
    };
    while (alive) {
      alive = wait_all(w_empty + 8 * slot, wphase ^ 1u);
      if (!alive) break;
      int it = 0;
      if (lane == 0) {
        it = atomicAdd(a.kv_counter, 1);
        if (it >= n_items) it = -1;
        sts_u32(w_item + 4 * slot, (uint32_t)it);
        mbar_arrive(w_full + 8 * slot);
      }
      it = __shfl_sync(0xffffffffu, it, 0);
      if (++slot == 2) { slot = 0; wphase ^= 1u; }
      if (it < 0) break;
      const int kt = it / n_bh, bh = it - kt * n_bh;
      const int b = bh / a.H, h = bh - b * a.H;
      int qt = __shfl_sync(0xffffffffu, next_marked(bh, first_q(kt)), 0);
      if (qt >= a.tiles_per_head) continue;            // no marked Q tile sees these keys
      alive = wait_all(kv_empty, kvphase ^ 1u);
      if (!alive) break;
      kvphase ^= 1u;
      if (elect_one()) {
        mbar_expect_tx(kv_full, 2 * C::kQBytes);
        for (int hf = 0; hf < C::kHalves; ++hf) {
          tma_load_4d(k_smem + hf * (TN * 128), &map_k, kv_full, hf * 64, kt * TN, h, b);
          tma_load_4d(v_smem + hf * (TN * 128), &map_v, kv_full, hf * 64, kt * TN, h, b);
        }
      }
      __syncwarp();
      while (qt < a.tiles_per_head && alive) {
        alive = wait_all(qdo_empty, qphase ^ 1u);
        if (!alive) break;
        qphase ^= 1u;
        if (elect_one()) {
          mbar_expect_tx(qdo_full, 2 * C::kQBytes);
          for (int hf = 0; hf < C::kHalves; ++hf) {
            tma_load_4d(q_smem + hf * (TM * 128), &map_q, qdo_full, hf * 64, qt * TM, h, b);
            tma_load_4d(do_smem + hf * (TM * 128), &map_do, qdo_full, hf * 64, qt * TM, h, b);
          }
        }
        __syncwarp();
        qt = __shfl_sync(0xffffffffu, next_marked(bh, qt + 1), 0);
      }
    }
    if (!alive && lane == 0) {
      bool ok = mbar_drain(qdo_full, qphase ^ 1u);
      ok &= mbar_drain(kv_full, kvphase ^ 1u);
      if (!ok) sts_u32(drain_fail, 1u);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    constexpr uint32_t id_kk = idesc_kk();
    constexpr uint32_t id_mn = idesc_mn<HD>();
    const uint64_t hi = (uint64_t)kDescHi << 32;
    const uint64_t q_d = hi | smem_desc_lo(q_smem), do_d = hi | smem_desc_lo(do_smem);
    const uint64_t k_d = hi | smem_desc_lo(k_smem), v_d = hi | smem_desc_lo(v_smem);
    const uint64_t q_n_d = hi | mn_desc_lo(q_smem), do_n_d = hi | mn_desc_lo(do_smem);
    const uint64_t ds_m_d = hi | mn_desc_lo(ds_smem), p_m_d = hi | mn_desc_lo(p_smem);
    uint32_t kvphase = 0, qphase = 0, sdphase = 0, pdsphase = 0, accphase = 0, wphase = 0;
    int slot = 0;
    bool alive = true;
    auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
    };
    while (alive) {
      alive = wait_all(w_full + 8 * slot, wphase);
      if (!alive) break;
      const int it = __shfl_sync(0xffffffffu, (int)lds_u32(w_item + 4 * slot), 0);
      __syncwarp();
      if (lane == 0) mbar_arrive(w_empty + 8 * slot);
      if (++slot == 2) { slot = 0; wphase ^= 1u; }
      if (it < 0) break;
      const int kt = it / n_bh, bh = it - kt * n_bh;
      int qt = __shfl_sync(0xffffffffu, next_marked(bh, first_q(kt)), 0);
      if (qt >= a.tiles_per_head) continue;
      alive = wait_all(kv_full, kvphase);
      kvphase ^= 1u;
      // the previous item's dK and dV must have been read before this item's first contraction overwrites them
      if (alive) alive = wait_all(acc_empty, accphase ^ 1u);
      accphase ^= 1u;
      if (!alive) break;
      bool first = true;
      while (qt < a.tiles_per_head && alive) {
        alive = wait_all(qdo_full, qphase);
        qphase ^= 1u;
        if (alive) alive = wait_all(sd_empty, sdphase ^ 1u);
        if (!alive) break;
        sdphase ^= 1u;
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int kk = 0; kk < HD / 16; ++kk) {
            const uint32_t off = (kk >> 2) * ((TM * 128) >> 4) + (kk & 3) * 2;
            umma_bf16_desc(tmem_base + C::kTmemS, q_d + off, k_d + off, id_kk, kk > 0 ? 1u : 0u);
          }
#pragma unroll
          for (int kk = 0; kk < HD / 16; ++kk) {
            const uint32_t off = (kk >> 2) * ((TM * 128) >> 4) + (kk & 3) * 2;
            umma_bf16_desc(tmem_base + C::kTmemDP, do_d + off, v_d + off, id_kk, kk > 0 ? 1u : 0u);
          }
          umma_commit(sd_full);
        }
        __syncwarp();
        // P and g dS of this pair are in shared memory
        alive = wait_all(pds_full, pdsphase);
        pdsphase ^= 1u;
        if (!alive) break;
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int kk = 0; kk < TM / 16; ++kk) {
            const uint32_t off = kk * ((16 * 128) >> 4);                             // 16 query rows
            umma_bf16_desc(tmem_base + kTmemDK, ds_m_d + off, q_n_d + off, id_mn, (!first || kk > 0) ? 1u : 0u);
          }
#pragma unroll
          for (int kk = 0; kk < TM / 16; ++kk) {
            const uint32_t off = kk * ((16 * 128) >> 4);
            umma_bf16_desc(tmem_base + kTmemDV, p_m_d + off, do_n_d + off, id_mn, (!first || kk > 0) ? 1u : 0u);
          }
          umma_commit(pds_empty);
          umma_commit(qdo_empty);
        }
        __syncwarp();
        first = false;
        qt = __shfl_sync(0xffffffffu, next_marked(bh, qt + 1), 0);
      }
      if (!alive) break;
      if (elect_one()) {
        umma_commit(acc_full);
        umma_commit(kv_empty);
      }
      __syncwarp();
    }
    if (!alive && lane == 0) {
      umma_commit(drain_bar);
      if (!mbar_drain(drain_bar, 0u)) sts_u32(drain_fail, 1u);
    }
  } else {
    // ------------------------------------------------------------------ consumers: four threads per TMEM lane
    const int quad = warp & 3;
    const int quarter = (warp - 2) >> 2;
    const int row_local = quad * 32 + lane;
    const uint32_t taddr_row = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint32_t sdphase = 0, pdsphase = 0, accphase = 0, wphase = 0, xphase = 0;
    int slot = 0;
    bool alive = true;
    while (alive) {
      alive = __all_sync(0xffffffffu, mbar_wait(w_full + 8 * slot, wphase, abort_flag));
      if (!alive) break;
      const int it = (int)lds_u32(w_item + 4 * slot);
      __syncwarp();
      if (lane == 0) mbar_arrive(w_empty + 8 * slot);
      if (++slot == 2) { slot = 0; wphase ^= 1u; }
      if (it < 0) break;
      const int kt = it / n_bh, bh = it - kt * n_bh;
      const int b = bh / a.H, h = bh - b * a.H;
      int qt = __shfl_sync(0xffffffffu, next_marked(bh, first_q(kt)), 0);
      if (qt >= a.tiles_per_head) continue;
      const float slope = a.alibi ? a.alibi[h] / a.sm_scale : 0.f;   // bias in accumulator units
      while (qt < a.tiles_per_head && alive) {
        // this thread's query row of the Q tile: TMEM lane = query row, as in the query-major pass
        const int i = qt * TM + row_local;
        const bool valid = i < a.N;
        const int id = bh * a.tiles_per_head + qt;
        const bool marked = valid && ((a.tile_mask[4 * (size_t)id + (row_local >> 5)] >> (row_local & 31)) & 1u);
        const size_t grow = (size_t)bh * a.N + (valid ? i : 0);
        const int lim = a.causal ? i : a.N - 1;
        const float c_i = valid ? a.scale[(size_t)b * a.scale_sb + (size_t)h * a.N + i] : 0.f;
        const float ra = a.alpha_m1 * (c_i * a.sm_scale);
        const float g = c_i * a.sm_scale;
        const float tau = marked ? a.tau[grow] : 0.f;
        const float rho = marked ? a.rho[grow] : 0.f;
        const float ra_m = marked ? ra : 0.f;
        alive = __all_sync(0xffffffffu, mbar_wait(sd_full, sdphase, abort_flag));
        if (!alive) break;
        sdphase ^= 1u;
        tc_fence_after();
        // P and dS of the previous pair must have been consumed before their buffers are rewritten
        alive = __all_sync(0xffffffffu, mbar_wait(pds_empty, pdsphase ^ 1u, abort_flag));
        pdsphase ^= 1u;
        if (!alive) break;
#pragma unroll 1
        for (int hc = 0; hc < 2; ++hc) {
          float sa[16], dp[16];
          tmem_ld16(taddr_row + C::kTmemS + quarter * 32 + hc * 16, sa);
          tmem_ld16(taddr_row + C::kTmemDP + quarter * 32 + hc * 16, dp);
          tmem_ld_wait();
          const int col0 = kt * TN + quarter * 32 + hc * 16;
          if (slope != 0.f) {
#pragma unroll
            for (int u = 0; u < 16; ++u) sa[u] = fmaf(slope, (float)(col0 + u - i), sa[u]);
          }
          const bool edge = col0 + 15 > lim;
          const uint32_t blk = (uint32_t)(quarter >> 1) * (TM * 128) + (uint32_t)row_local * 128u;
#pragma unroll
          for (int u4 = 0; u4 < 2; ++u4) {
            float pv[8], dv[8];
            if (EC != kExpoGeneral && !edge) {
              // away from the mask (an unmarked row has a = 0, tau = 0 here: every entry clamps to zero)
#pragma unroll
              for (int z = 0; z < 8; ++z) {
                const int u = u4 * 8 + z;
                const float m = fmaxf(fmaf(ra_m, sa[u], -tau), 0.f);
                const float ye1 = clamped_pow_m1<EC>(m);
                pv[z] = ye1 * m;
                dv[z] = g * (ye1 * (dp[u] - rho));
              }
            } else {
#pragma unroll
              for (int z = 0; z < 8; ++z) {
                const int u = u4 * 8 + z;
                const float yr = fmaf(ra, sa[u], -tau);
                const bool ok = marked && yr > 0.f && (!edge || col0 + u <= lim);
                float ye, ye1;
                pow_pair_c<EC>(ok ? yr : 0.f, ok, a.expo, ye, ye1);
                pv[z] = ye;
                dv[z] = g * (ye1 * (dp[u] - rho));
              }
            }
            const uint32_t unit = (uint32_t)((quarter & 1) * 4 + hc * 2 + u4);
            const uint32_t off = blk + ((unit ^ (uint32_t)(row_local & 7)) << 4);
            asm volatile("st.shared::cta.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(p_smem + off),
                         "r"(pack_bf16(pv[0], pv[1])), "r"(pack_bf16(pv[2], pv[3])), "r"(pack_bf16(pv[4], pv[5])),
                         "r"(pack_bf16(pv[6], pv[7]))
                         : "memory");
            asm volatile("st.shared::cta.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(ds_smem + off),
                         "r"(pack_bf16(dv[0], dv[1])), "r"(pack_bf16(dv[2], dv[3])), "r"(pack_bf16(dv[4], dv[5])),
                         "r"(pack_bf16(dv[6], dv[7]))
                         : "memory");
          }
        }
        tc_fence_before();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(sd_empty);
          mbar_arrive(pds_full);
        }
        qt = __shfl_sync(0xffffffffu, next_marked(bh, qt + 1), 0);
      }
      if (!alive) break;
      // ---- dK and dV of the K tile: TMEM lane = key; through a staging tile (the P and g dS buffers, free once the
      //      item's last contraction has finished) and bulk tensor reductions into the fp32 accumulators
      alive = __all_sync(0xffffffffu, mbar_wait(acc_full, accphase, abort_flag));
      accphase ^= 1u;
      if (!alive) break;
      tc_fence_after();
      const int key0 = kt * TN;
#pragma unroll 1
      for (int which = 0; which < 2 && alive; ++which) {
        if (quarter < HD / 32) {
          float va[32];
          tmem_ld32(taddr_row + (which == 0 ? kTmemDK : kTmemDV) + quarter * 32, va);
          tmem_ld_wait();
          const uint32_t dst = p_smem + (uint32_t)quarter * (TM * 128) + (uint32_t)row_local * 128u;
#pragma unroll
          for (int u = 0; u < 8; ++u)
            asm volatile("st.shared::cta.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (((uint32_t)u ^ (uint32_t)(row_local & 7)) << 4)),
                         "f"(va[4 * u]), "f"(va[4 * u + 1]), "f"(va[4 * u + 2]), "f"(va[4 * u + 3])
                         : "memory");
        }
        tc_fence_before();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          if (which == 1) mbar_arrive(acc_empty);      // both accumulators are out of TMEM
          mbar_arrive(x_bar);
        }
        alive = __all_sync(0xffffffffu, mbar_wait(x_bar, xphase, abort_flag));
        xphase ^= 1u;
        if (!alive) break;
        if (threadIdx.x == 64) {
          const CUtensorMap* map = which == 0 ? &map_dk : &map_dv;
#pragma unroll
          for (int c = 0; c < HD / 32; ++c)
            asm volatile(
                "cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(
                    reinterpret_cast<uint64_t>(map)),
                "r"(p_smem + (uint32_t)c * (TM * 128)), "r"(c * 32), "r"(key0), "r"(bh)
                : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(x_bar);
        alive = __all_sync(0xffffffffu, mbar_wait(x_bar, xphase, abort_flag));
        xphase ^= 1u;
      }
    }
    if (threadIdx.x == 64) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (lds_u32(abort_flag)) {
    if (threadIdx.x == 0 && a.status) atomicOr(a.status + ENTMAX_ATTN_STATUS_FLAGS, ENTMAX_ATTN_FLAG_WAIT_EXPIRED);
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

template <int HD, int EC>
cudaError_t launch_tile_bwd_impl(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                                 const TileBwdArgs& args, cudaStream_t stream) {
  CUtensorMap map_q, map_k, map_v, map_do;
  cudaError_t err = make_tile_map(&map_q, q, p.D, p.N, p.H, p.B, p.sn, p.sh, p.sb);
  if (err != cudaSuccess) return err;
  err = make_tile_map(&map_k, k, p.D, p.N, p.H, p.B, p.sn, p.sh, p.sb);
  if (err != cudaSuccess) return err;
  err = make_tile_map(&map_v, v, p.D, p.N, p.H, p.B, p.sn, p.sh, p.sb);
  if (err != cudaSuccess) return err;
  err = make_tile_map(&map_do, d_o, p.D, p.N, p.H, p.B, p.sn, p.sh, p.sb);
  if (err != cudaSuccess) return err;
  CUtensorMap map_dk, map_dv;
  err = make_acc_map(&map_dk, args.acc_dk, p.D, p.N, p.B * p.H);
  if (err != cudaSuccess) return err;
  err = make_acc_map(&map_dv, args.acc_dv, p.D, p.N, p.B * p.H);
  if (err != cudaSuccess) return err;
  err = cudaFuncSetAttribute(tile_bwd_kernel<HD, EC>, cudaFuncAttributeMaxDynamicSharedMemorySize, BCfg<HD>::kSmemBytes);
  if (err != cudaSuccess) return err;
  int dev = 0, sms = 0;
  err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;
  const long all_tiles = (long)p.B * p.H * args.tiles_per_head;
  const int grid = (int)(all_tiles < sms ? all_tiles : sms);
  tile_bwd_kernel<HD, EC><<<grid, kThreadsB, BCfg<HD>::kSmemBytes, stream>>>(map_q, map_k, map_v, map_do, args);
  err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  // dK and dV of the same Q tiles, key-major (needs the rho the kernel above leaves behind)
  err = cudaFuncSetAttribute(tile_bwd_kv_kernel<HD, EC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             BCfg<HD>::kSmemBytes);
  if (err != cudaSuccess) return err;
  tile_bwd_kv_kernel<HD, EC><<<grid, kThreadsB, BCfg<HD>::kSmemBytes, stream>>>(map_q, map_k, map_v, map_do, map_dk,
                                                                                map_dv, args);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_tile_bwd(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                            const float* scale, const float* tau, const int32_t* row_list, const int32_t* row_count,
                            uint32_t* tile_mask, int32_t* tile_flag, int32_t* tile_list, int32_t* tile_count,
                            int32_t* work_counter, float* rho, void* dq, float* acc_dk, float* acc_dv, float* dc_rows,
                            int32_t* status, cudaStream_t stream) {
  const int tiles_per_head = (p.N + TM - 1) / TM;
  mark_tiles_kernel<<<148, 256, 0, stream>>>(p.N, tiles_per_head, row_list, row_count, tile_mask, tile_flag, tile_list,
                                             tile_count);
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  err = order_tiles(p, tile_flag, tile_list, tile_count, stream);
  if (err != cudaSuccess) return err;
  TileBwdArgs args;
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
  args.kv_counter = work_counter + 12;   // (the counter block's last word)
  args.tile_flag = tile_flag;
  args.rho = rho;
  args.tile_mask = tile_mask;
  args.tau = tau;
  args.dq = dq;
  args.acc_dk = acc_dk;
  args.acc_dv = acc_dv;
  args.dc_rows = dc_rows;
  args.sb = p.sb; args.sh = p.sh; args.sn = p.sn;
  args.status = status;
  args.tiles_per_head = tiles_per_head;
#define ENTMAX_TILE_BWD(EC)                                                                 \
  (p.D == 64 ? launch_tile_bwd_impl<64, EC>(p, q, k, v, d_o, args, stream)                   \
             : launch_tile_bwd_impl<128, EC>(p, q, k, v, d_o, args, stream))
  switch (p.expo_class) {
    case kExpo2: return ENTMAX_TILE_BWD(kExpo2);
    case kExpo1: return ENTMAX_TILE_BWD(kExpo1);
    case kExpo4: return ENTMAX_TILE_BWD(kExpo4);
    default: return ENTMAX_TILE_BWD(kExpoGeneral);
  }
#undef ENTMAX_TILE_BWD
}

}  // namespace entmax
