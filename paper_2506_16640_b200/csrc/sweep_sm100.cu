// Score sweep for bf16 problems on sm_100a: S = Q K^T on tcgen05 tensor cores (bf16 in, fp32
// accumulators in TMEM, Q and K tiles staged by TMA without multicast), one pass over the keys of
// every query row, leaving a short per-row candidate list that provably contains the support of
// Eq. 1.
//
// Why one pass is enough.  Write y_j = (alpha-1) s_ij and f(tau) = sum_j [y_j - tau]_+^e - 1, e = 1/(alpha-1).
//  (1) p_max <= 1 gives tau >= y_max - 1 (lower end of the bracket of App. A), and
//  (2) the threshold of a prefix of the row never exceeds the threshold of the whole row (adding a
//      logit never lowers tau), while keys at or below the threshold do not change it.
// So while the keys stream by, each row keeps a lower bound thr on its final tau and the list of keys
// seen so far with y > thr.  When the list fills up, a few Newton steps on the listed keys, started
// at thr, raise thr (f is convex and decreasing for e >= 1, so Newton from the left of the root never
// passes it) and the list is filtered.  A row whose list cannot be kept below kListKeep entries is
// flagged and later recomputed by the dense-row path.  In backward mode the threshold is the tau of
// the forward pass and the list is simply the support.
//
// CTA layout (320 threads, one CTA per SM, persistent over work units):
//   warp 0        TMA producer: Q tile pair (2 x 128 rows) once per item, K tiles of BN keys through a ring
//   warp 1        MMA issuer: per K tile two M=128 x N=BN accumulations (one per Q tile) into TMEM
//   warps 2..5    consumer group 0: TMEM lane = query row of Q tile 0, one thread per row
//   warps 6..9    consumer group 1: same for Q tile 1
// Every mbarrier wait is bounded: on expiry the CTA raises ENTMAX_ATTN_FLAG_WAIT_EXPIRED, all roles
// leave their loops, in-flight copies are given time to land, TMEM is freed and the CTA returns.
#include <cuda.h>

#include "common.cuh"

namespace entmax {

namespace {

constexpr int BM = 128;          // query rows per Q tile = TMEM lanes
constexpr int BN = 256;          // keys per K tile = N of one MMA
constexpr int kQTiles = 2;       // Q tiles per item
constexpr int kItemRows = BM * kQTiles;
constexpr int kThreads = 320;
constexpr int kTmemCols = 512;
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s

template <int HD>
struct Cfg {
  static constexpr int kHalves = HD / 64;                 // 64 bf16 = one 128-byte swizzle row
  static constexpr int kQBytes = BM * HD * 2;
  static constexpr int kKBytes = BN * HD * 2;
  static constexpr int kStages = HD == 128 ? 2 : 4;
  static constexpr int kSmemBytes = kQTiles * kQBytes + kStages * kKBytes + 1024 /*align*/ + 256 /*barriers*/;
};

struct SweepArgs {
  int B, H, N;
  int causal;
  int mode;             // 0: search the threshold; 1: threshold given (tau_in)
  int expo_class;
  float expo;
  float alpha_m1;       // alpha - 1
  float sm_scale;
  const float* scale;   // [H, N]
  const float* tau_in;  // [B*H*N] (mode 1)
  int32_t* row_cnt;
  float* row_thr;
  Entry* entries;
  float* dump;          // optional [N, N] raw accumulators of head dump_bh
  int dump_bh;
  int32_t* status;
  int items_per_bh;     // ceil(N / kItemRows)
  int units_per_bh;
  int n_units;
};

// ------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      " .reg .pred p;\n"
      " mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      " selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when the CTA is aborting (this or another wait ran out of time).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  uint32_t spins = 0;
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 63u) == 0u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 x bf16 -> fp32, issued by one thread
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n"
      " .reg .pred p;\n"
      " setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// mbarrier arrive once every MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread t of the warp gets lane (base + t)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&r)[32]) {
  uint32_t* u = reinterpret_cast<uint32_t*>(r);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]),
        "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]),
        "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]),
        "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, K-major operand, 128-byte swizzle: rows are 128 bytes apart, groups
// of 8 rows 1024 bytes apart (stride-dimension offset); descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;                 // leading-dimension offset: not used by swizzled K-major layouts
  d |= (uint64_t)(1024 >> 4) << 32;       // stride-dimension offset
  d |= (uint64_t)1 << 46;                 // descriptor version
  d |= (uint64_t)2 << 61;                 // 128-byte swizzle
  return d;
}
// Instruction descriptor: fp32 accumulate, A and B bf16, both K-major, M = 128, N = BN
__host__ __device__ constexpr uint32_t make_idesc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// --------------------------------------------------------------------------------- work schedule
// Unit u of head-pair bh: causal -> items (long, short) = (n-1-w, w) so that every unit costs the same;
// non-causal -> one item.  Returns the number of items (1 or 2).
__device__ __forceinline__ int unit_items(const SweepArgs& a, int unit, int& bh, int (&item)[2]) {
  bh = unit / a.units_per_bh;
  const int w = unit - bh * a.units_per_bh;
  if (!a.causal) { item[0] = w; return 1; }
  item[0] = a.items_per_bh - 1 - w;
  item[1] = w;
  return item[0] == item[1] ? 1 : 2;
}
__device__ __forceinline__ int item_tiles(const SweepArgs& a, int item) {
  if (!a.causal) return (a.N + BN - 1) / BN;
  int last_row = item * kItemRows + kItemRows - 1;
  if (last_row > a.N - 1) last_row = a.N - 1;
  return last_row / BN + 1;
}

// ------------------------------------------------------------------------------- per-row state
struct RowState {
  float thr_acc;   // candidates are accumulators above this
  float m_run;     // running maximum accumulator
  float a, inv_a;  // y = a * acc
  int cnt;         // list length; -1 = handed to the dense path
  int lim;         // largest visible key index
  Entry* list;
};

__device__ __noinline__ void shrink_list(RowState& r, int mode, int expo_class, float expo) {
  if (mode != 0) {  // threshold given: a full list means the support does not fit
    r.cnt = -1;
    r.thr_acc = INFINITY;
    return;
  }
  float tau = r.thr_acc * r.a;
  for (int it = 0; it < 3; ++it) {
    float s0 = 0.f, s1 = 0.f;
    for (int t = 0; t < r.cnt; ++t) {
      const float y = fmaf(r.a, r.list[t].y, -tau);
      if (y > 0.f) {
        float ye, ye1;
        pow_pair(y, expo_class, expo, ye, ye1);
        s0 += ye;
        s1 += ye1;
      }
    }
    if (!(s0 > 1.0f) || !(s1 > 0.f)) break;
    tau += (s0 - 1.0f) / (expo * s1);
  }
  const float thr = fmaxf(r.thr_acc, tau * r.inv_a);
  int kept = 0;
  for (int t = 0; t < r.cnt; ++t) {
    const Entry e = r.list[t];
    if (e.y > thr) r.list[kept++] = e;
  }
  r.thr_acc = thr;
  r.cnt = kept;
  if (kept > kListKeep) {
    r.cnt = -1;
    r.thr_acc = INFINITY;
  }
}

__device__ __forceinline__ void push(RowState& r, float acc, int j, int mode, int expo_class, float expo) {
  r.list[r.cnt].y = acc;
  r.list[r.cnt].j = j;
  if (++r.cnt == kListCap) shrink_list(r, mode, expo_class, expo);
}

// One 32-column chunk of a score tile for this thread's row.
template <bool kMasked>
__device__ __forceinline__ void scan_chunk(float (&v)[32], int col0, RowState& r, int mode, int expo_class, float expo) {
  if (kMasked) {
#pragma unroll
    for (int t = 0; t < 32; ++t) v[t] = (col0 + t <= r.lim) ? v[t] : -INFINITY;
  }
  float m = max3(v[0], v[1], v[2]);
#pragma unroll
  for (int t = 3; t < 31; t += 2) m = max3(m, v[t], v[t + 1]);
  m = fmaxf(m, v[31]);
  if (m > r.thr_acc) {
    if (mode == 0) {
      r.m_run = fmaxf(r.m_run, m);
      r.thr_acc = fmaxf(r.thr_acc, r.m_run - r.inv_a);
    }
#pragma unroll
    for (int t = 0; t < 32; ++t) {
      if (v[t] > r.thr_acc) push(r, v[t], col0 + t, mode, expo_class, expo);
    }
  }
}

template <int HD>
__global__ void __launch_bounds__(kThreads, 1) sweep_kernel(const __grid_constant__ CUtensorMap map_q,
                                                            const __grid_constant__ CUtensorMap map_k,
                                                            const SweepArgs a) {
  using C = Cfg<HD>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_smem = smem;                                   // [kQTiles][kHalves][BM rows x 128 B]
  uint8_t* k_smem = smem + kQTiles * C::kQBytes;            // [kStages][kHalves][BN rows x 128 B]
  uint64_t* bars = reinterpret_cast<uint64_t*>(k_smem + C::kStages * C::kKBytes);
  uint64_t* q_full = bars;                  // [2]
  uint64_t* q_empty = bars + 2;             // [2]
  uint64_t* s_full = bars + 4;              // [2]
  uint64_t* s_empty = bars + 6;             // [2]
  uint64_t* k_full = bars + 8;              // [kStages]
  uint64_t* k_empty = bars + 8 + C::kStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8 + 2 * C::kStages);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int t = 0; t < 2; ++t) {
      mbar_init(&q_full[t], 1);
      mbar_init(&q_empty[t], 1);
      mbar_init(&s_full[t], 1);
      mbar_init(&s_empty[t], BM);
    }
    for (int t = 0; t < C::kStages; ++t) {
      mbar_init(&k_full[t], 1);
      mbar_init(&k_empty[t], 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t kphase = 0, qphase = 0;
      bool alive = true;
      for (int unit = blockIdx.x; unit < a.n_units && alive; unit += gridDim.x) {
        int bh, item[2];
        const int n_items = unit_items(a, unit, bh, item);
        const int b = bh / a.H, h = bh - b * a.H;
        for (int s = 0; s < n_items && alive; ++s) {
          const int tiles = item_tiles(a, item[s]);
          for (int t = 0; t < tiles && alive; ++t) {
            alive = mbar_wait(&k_empty[stage], kphase ^ 1u, abort_flag);
            if (!alive) break;
            mbar_expect_tx(&k_full[stage], C::kKBytes);
            for (int hf = 0; hf < C::kHalves; ++hf)
              tma_load_4d(k_smem + stage * C::kKBytes + hf * (BN * 128), &map_k, &k_full[stage], hf * 64, t * BN, h, b);
            if (++stage == C::kStages) { stage = 0; kphase ^= 1u; }
            if (t == 0) {
              for (int x = 0; x < kQTiles && alive; ++x) {
                alive = mbar_wait(&q_empty[x], qphase ^ 1u, abort_flag);
                if (!alive) break;
                mbar_expect_tx(&q_full[x], C::kQBytes);
                for (int hf = 0; hf < C::kHalves; ++hf)
                  tma_load_4d(q_smem + x * C::kQBytes + hf * (BM * 128), &map_q, &q_full[x], hf * 64,
                              item[s] * kItemRows + x * BM, h, b);
              }
              qphase ^= 1u;
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc();
      int stage = 0;
      uint32_t kphase = 0, qphase = 0, sphase[2] = {0, 0};
      bool alive = true;
      for (int unit = blockIdx.x; unit < a.n_units && alive; unit += gridDim.x) {
        int bh, item[2];
        const int n_items = unit_items(a, unit, bh, item);
        for (int s = 0; s < n_items && alive; ++s) {
          const int tiles = item_tiles(a, item[s]);
          for (int t = 0; t < tiles && alive; ++t) {
            alive = mbar_wait(&k_full[stage], kphase, abort_flag);
            if (!alive) break;
            const uint32_t kaddr = smem_u32(k_smem + stage * C::kKBytes);
            for (int x = 0; x < kQTiles && alive; ++x) {
              if (t == 0) alive = mbar_wait(&q_full[x], qphase, abort_flag);
              if (alive) alive = mbar_wait(&s_empty[x], sphase[x] ^ 1u, abort_flag);
              if (!alive) break;
              sphase[x] ^= 1u;
              tc_fence_after();
              const uint32_t qaddr = smem_u32(q_smem + x * C::kQBytes);
#pragma unroll
              for (int kk = 0; kk < HD / 16; ++kk) {
                const uint32_t hf = kk >> 2, within = (kk & 3) * 32;
                umma_bf16(tmem_base + x * BN, smem_desc_sw128(qaddr + hf * (BM * 128) + within),
                          smem_desc_sw128(kaddr + hf * (BN * 128) + within), idesc, kk > 0 ? 1u : 0u);
              }
              umma_commit(&s_full[x]);
              if (t == tiles - 1) umma_commit(&q_empty[x]);
            }
            if (!alive) break;
            umma_commit(&k_empty[stage]);
            if (++stage == C::kStages) { stage = 0; kphase ^= 1u; }
          }
          qphase ^= 1u;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers: one thread per query row
    const int x = (warp - 2) >> 2;                 // Q tile of this group
    const int quad = warp & 3;                     // TMEM lane quadrant this warp may read
    const int row_local = quad * 32 + lane;
    const uint32_t taddr_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(x * BN);
    uint32_t fphase = 0;
    bool alive = true;
    for (int unit = blockIdx.x; unit < a.n_units && alive; unit += gridDim.x) {
      int bh, item[2];
      const int n_items = unit_items(a, unit, bh, item);
      const int h = bh % a.H;
      for (int s = 0; s < n_items && alive; ++s) {
        const int tiles = item_tiles(a, item[s]);
        const int tile_row0 = item[s] * kItemRows + x * BM;
        const int i = tile_row0 + row_local;
        const bool valid = i < a.N;
        const size_t grow = (size_t)bh * a.N + (valid ? i : 0);
        RowState r;
        r.list = a.entries + grow * kListCap;
        r.cnt = 0;
        r.m_run = -INFINITY;
        r.lim = a.causal ? i : a.N - 1;
        r.thr_acc = INFINITY;
        r.a = 1.f;
        r.inv_a = 1.f;
        if (valid) {
          r.a = a.alpha_m1 * (a.scale[(size_t)h * a.N + i] * a.sm_scale);
          if (r.a > 0.f && r.a < INFINITY) {
            r.inv_a = 1.0f / r.a;
            if (a.mode == 0) {
              r.thr_acc = -INFINITY;
            } else {
              const float t_acc = a.tau_in[grow] * r.inv_a;
              r.thr_acc = t_acc - 1e-6f * fabsf(t_acc);   // a hair below: the row kernel applies the exact test
            }
          } else {
            r.cnt = -1;   // non-positive or non-finite scale: dense path
          }
        }
        const bool dump_here = a.dump != nullptr && bh == a.dump_bh && valid;
        // tiles that reach past the last visible key of this Q tile's first row need the mask
        const int first_lim = a.causal ? tile_row0 : a.N - 1;
        for (int t = 0; t < tiles && alive; ++t) {
          // the warp leaves together: tcgen05.ld needs all 32 lanes
          alive = __all_sync(0xffffffffu, mbar_wait(&s_full[x], fphase, abort_flag));
          if (!alive) break;
          fphase ^= 1u;
          tc_fence_after();
          const bool masked = t * BN + BN - 1 > first_lim;
#pragma unroll 1
          for (int c = 0; c < BN / 32; ++c) {
            float v[32];
            __syncwarp();
            tmem_ld32(taddr_row + c * 32, v);
            tmem_ld_wait();
            const int col0 = t * BN + c * 32;
            if (dump_here) {
              for (int u = 0; u < 32; ++u)
                if (col0 + u <= r.lim) a.dump[(size_t)i * a.N + col0 + u] = v[u];
            }
            if (masked) scan_chunk<true>(v, col0, r, a.mode, a.expo_class, a.expo);
            else scan_chunk<false>(v, col0, r, a.mode, a.expo_class, a.expo);
          }
          tc_fence_before();
          mbar_arrive(&s_empty[x]);
        }
        if (valid && alive) {
          a.row_cnt[grow] = r.cnt;
          a.row_thr[grow] = r.thr_acc * r.a;
        }
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0 && a.status) atomicOr(a.status + ENTMAX_ATTN_STATUS_FLAGS, ENTMAX_ATTN_FLAG_WAIT_EXPIRED);
    // give copies and MMAs that may still be in flight time to land before shared memory and TMEM go away
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < 200000ull) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
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

template <int HD>
cudaError_t launch_impl(const Problem& p, const void* q, const void* k, SweepArgs& args, cudaStream_t stream) {
  CUtensorMap map_q, map_k;
  cudaError_t err = make_map(&map_q, q, p, BM);
  if (err != cudaSuccess) return err;
  err = make_map(&map_k, k, p, BN);
  if (err != cudaSuccess) return err;
  err = cudaFuncSetAttribute(sweep_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<HD>::kSmemBytes);
  if (err != cudaSuccess) return err;
  int dev = 0, sms = 0;
  err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;
  const int grid = args.n_units < sms ? args.n_units : sms;
  sweep_kernel<HD><<<grid, kThreads, Cfg<HD>::kSmemBytes, stream>>>(map_q, map_k, args);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_sweep(const Problem& p, const void* q, const void* k, const float* scale, const float* tau_in,
                         int mode, int32_t* row_cnt, float* row_thr, Entry* entries, float* dump, int dump_bh,
                         int32_t* status, cudaStream_t stream) {
  SweepArgs args;
  args.B = p.B; args.H = p.H; args.N = p.N;
  args.causal = p.causal;
  args.mode = mode;
  args.expo_class = p.expo_class;
  args.expo = p.expo;
  args.alpha_m1 = p.alpha - 1.0f;
  args.sm_scale = p.sm_scale;
  args.scale = scale;
  args.tau_in = tau_in;
  args.row_cnt = row_cnt;
  args.row_thr = row_thr;
  args.entries = entries;
  args.dump = dump;
  args.dump_bh = dump_bh;
  args.status = status;
  args.items_per_bh = (p.N + kItemRows - 1) / kItemRows;
  args.units_per_bh = p.causal ? (args.items_per_bh + 1) / 2 : args.items_per_bh;
  args.n_units = args.units_per_bh * p.B * p.H;
  return p.D == 64 ? launch_impl<64>(p, q, k, args, stream) : launch_impl<128>(p, q, k, args, stream);
}

}  // namespace entmax
