// Decode-shape score stream on sm_100a.  With a handful of query rows the products q.k are still a
// contraction over the head dimension; done with FMAs they cost 8 * q_len instructions per 16 bytes of
// K, which outruns HBM once q_len > 2.  Here the K tile is the M side of the MMA instead:
//   D[128 keys, 16] = K_tile[128 keys, d] * Qpad[16, d]^T      (tcgen05, bf16 in, fp32 in TMEM)
// with the q_len query rows zero-padded to 16 (the smallest N for M = 128).  TMEM lane = key, column =
// query: afterwards one thread owns one key and writes its q_len scores y = a_t (acc + bias), coalesced
// along the keys.  K arrives by TMA through a three-stage ring (96 KB of loads in flight per CTA, two
// CTAs per SM), so the kernel runs at the speed K can be read from HBM.
//
// CTA: warp 0 TMA producer, warp 1 MMA issuer, warps 2..5 one thread per key of the tile.  A CTA takes
// chunk_keys consecutive keys of one (sequence, head).  Every wait is bounded (sm100_ptx.cuh).
#include <cuda.h>

#include "decode.cuh"
#include "sm100_ptx.cuh"

namespace entmax {

namespace {

using namespace sm100;

constexpr int kTile = 128;         // keys per MMA tile = TMEM lanes
constexpr int kQPad = 16;          // query rows padded to the MMA's N
constexpr int kStagesD = 3;
constexpr int kThreadsD = 6 * 32;

template <int HD>
struct DCfg {
  static constexpr int kHalves = HD / 64;
  static constexpr int kKBytes = kTile * HD * 2;
  static constexpr int kQBytes = kQPad * HD * 2;
  static constexpr int kBarBytes = 128;
  static constexpr int kSmemBytes = kStagesD * kKBytes + kQBytes + 1024 + kBarBytes;
};

// A = K tile, B = padded Q, both K-major bf16, fp32 accumulate, M = 128, N = 16
__host__ __device__ constexpr uint32_t idesc_kq() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kQPad >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);
}

template <int HD>
__global__ void __launch_bounds__(kThreadsD, 2) decode_scores_tc_kernel(const __grid_constant__ CUtensorMap map_q,
                                                                       const __grid_constant__ CUtensorMap map_k,
                                                                       const DecodeArgs a,
                                                                       float* __restrict__ scores,
                                                                       float* __restrict__ chunk_max,
                                                                       int32_t* __restrict__ status) {
  using C = DCfg<HD>;
  extern __shared__ uint8_t smem_raw[];
  __shared__ float smax[4][ENTMAX_ATTN_DECODE_MAX_Q];
  const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int len = seq_len(a, b, status);
  const int key0 = chunk * a.chunk_keys;
  if (key0 >= len) return;                                  // whole CTA: nothing allocated yet
  int tiles = a.chunk_keys / kTile;
  const int left = (len - key0 + kTile - 1) / kTile;
  if (left < tiles) tiles = left;

  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t k_smem = sbase;                            // [kStagesD] K tiles
  const uint32_t q_smem = k_smem + kStagesD * C::kKBytes;
  const uint32_t bars = q_smem + C::kQBytes;
  const uint32_t q_full = bars;
  const uint32_t kv_full = bars + 8;                        // [kStagesD]
  const uint32_t kv_empty = kv_full + 8 * kStagesD;         // [kStagesD]
  const uint32_t s_full = kv_empty + 8 * kStagesD;          // [2]
  const uint32_t s_empty = s_full + 16;                     // [2]
  const uint32_t tmem_slot = s_empty + 16;
  const uint32_t abort_flag = tmem_slot + 4;
  const uint32_t drain_bar = tmem_slot + 8;       // teardown: every MMA issued so far has finished
  const uint32_t drain_fail = drain_bar + 8;      // uint32: a teardown wait ran out as well
  static_assert(8 * (1 + 2 * kStagesD + 4) + 8 + 16 <= C::kBarBytes, "barrier area");

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < kStagesD; ++s) {
      mbar_init(kv_full + 8 * s, 1);
      mbar_init(kv_empty + 8 * s, 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(s_full + 8 * s, 1);
      mbar_init(s_empty + 8 * s, 4);
    }
    mbar_init(drain_bar, 1);
    sts_u32(drain_fail, 0u);
    sts_u32(abort_flag, 0u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 32);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = lds_u32(tmem_slot);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(q_full, C::kQBytes);
      for (int hf = 0; hf < C::kHalves; ++hf) tma_load_4d(q_smem + hf * (kQPad * 128), &map_q, q_full, hf * 64, 0, h, b);
      int stage = 0;
      uint32_t phase = 0;
      bool alive = true;
      for (int t = 0; t < tiles; ++t) {
        alive = mbar_wait(kv_empty + 8 * stage, phase ^ 1u, abort_flag);
        if (!alive) break;
        mbar_expect_tx(kv_full + 8 * stage, C::kKBytes);
        for (int hf = 0; hf < C::kHalves; ++hf)
          tma_load_4d(k_smem + stage * C::kKBytes + hf * (kTile * 128), &map_k, kv_full + 8 * stage, hf * 64,
                      key0 + t * kTile, h, b);
        if (++stage == kStagesD) { stage = 0; phase ^= 1u; }
      }
      if (!alive) {
        // a wait ran out somewhere in the CTA: the copies this thread armed barriers for must land before shared
        // memory goes away (stages before `stage`: this round of the ring; the others: the previous round)
        bool ok = mbar_drain(q_full, 0u);
        for (int st = 0; st < kStagesD; ++st) ok &= mbar_drain(kv_full + 8 * st, st < stage ? phase : phase ^ 1u);
        if (!ok) sts_u32(drain_fail, 1u);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_kq();
      const uint32_t k_lo = smem_desc_lo(k_smem), q_lo = smem_desc_lo(q_smem);
      int stage = 0, buf = 0;
      uint32_t phase = 0, sphase[2] = {0, 0};
      bool alive = mbar_wait(q_full, 0, abort_flag);
      for (int t = 0; t < tiles && alive; ++t) {
        alive = mbar_wait(kv_full + 8 * stage, phase, abort_flag);
        if (alive) alive = mbar_wait(s_empty + 8 * buf, sphase[buf] ^ 1u, abort_flag);
        if (!alive) break;
        sphase[buf] ^= 1u;
        tc_fence_after();
        const uint32_t a_lo = k_lo + stage * (C::kKBytes >> 4);
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          const uint32_t a_off = (kk >> 2) * ((kTile * 128) >> 4) + (kk & 3) * 2;
          const uint32_t b_off = (kk >> 2) * ((kQPad * 128) >> 4) + (kk & 3) * 2;
          umma_bf16(tmem_base + buf * kQPad, a_lo + a_off, q_lo + b_off, kDescHi, idesc, kk > 0 ? 1u : 0u);
        }
        umma_commit(s_full + 8 * buf);
        umma_commit(kv_empty + 8 * stage);
        buf ^= 1;
        if (++stage == kStagesD) { stage = 0; phase ^= 1u; }
      }
      if (!alive) {
        // the tensor core must be done with shared memory and TMEM before they are released
        umma_commit(drain_bar);
        if (!mbar_drain(drain_bar, 0u)) sts_u32(drain_fail, 1u);
      }
    }
  } else {
    // ------------------------------------------------------------------ one thread per key of the tile
    const int quad = warp & 3;
    const int row_local = quad * 32 + lane;
    const uint32_t taddr_row = tmem_base + ((uint32_t)(quad * 32) << 16);
    const int bh = b * a.H + h;
    const int pos0 = len - a.QL;                                   // position of query 0
    const float slope = a.alibi ? a.alibi[h] / a.sm_scale : 0.f;   // bias in dot-product units
    // a_t = (alpha-1) c_t sm_scale with c_t = delta + beta (ln n_t)^gamma, n_t = pos_t + 1 (c_t = delta for
    // n_t = 1; 1 without scale parameters): lane t evaluates it in fp32 and the warp shares the values
    float a_lane = 0.f;
    if (lane < a.QL) {
      float c = 1.0f;
      if (a.beta) {
        const int n = pos0 + lane + 1;
        c = a.delta[h];
        if (n > 1) c += a.beta[h] * powf(logf((float)n), a.gamma[h]);
        if (!isfinite(c) && status) atomicOr(status + ENTMAX_ATTN_STATUS_FLAGS, ENTMAX_ATTN_FLAG_BAD_SCALE);
      }
      a_lane = a.alpha_m1 * (c * a.sm_scale);
    }
    float at[ENTMAX_ATTN_DECODE_MAX_Q], vmax[ENTMAX_ATTN_DECODE_MAX_Q];
#pragma unroll
    for (int t = 0; t < ENTMAX_ATTN_DECODE_MAX_Q; ++t) {
      at[t] = __shfl_sync(0xffffffffu, a_lane, t);
      vmax[t] = -INFINITY;
    }
    uint32_t sphase[2] = {0, 0};
    int buf = 0;
    bool alive = true;
    for (int t = 0; t < tiles && alive; ++t) {
      alive = __all_sync(0xffffffffu, mbar_wait(s_full + 8 * buf, sphase[buf], abort_flag));
      if (!alive) break;
      sphase[buf] ^= 1u;
      tc_fence_after();
      float acc[8];
      tmem_ld8(taddr_row + buf * kQPad, acc);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s_empty + 8 * buf);
      buf ^= 1;
      const int j = key0 + t * kTile + row_local;
      if (j < len) {
#pragma unroll
        for (int tq = 0; tq < ENTMAX_ATTN_DECODE_MAX_Q; ++tq) {
          if (tq < a.QL) {
            const int pos = pos0 + tq;
            const float y = j <= pos ? at[tq] * fmaf(slope, (float)(j - pos), acc[tq]) : -INFINITY;
            scores[((size_t)bh * a.QL + tq) * a.score_stride + j] = y;
            vmax[tq] = fmaxf(vmax[tq], y);
          }
        }
      }
    }
    // chunk maximum per query: the warp, then the four warps
#pragma unroll
    for (int tq = 0; tq < ENTMAX_ATTN_DECODE_MAX_Q; ++tq) {
      float m = vmax[tq];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      if (lane == 0) smax[quad][tq] = m;
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (alive && row_local < a.QL) {
      const float m = fmaxf(fmaxf(smax[0][row_local], smax[1][row_local]), fmaxf(smax[2][row_local], smax[3][row_local]));
      chunk_max[((size_t)bh * a.QL + row_local) * a.n_chunks + chunk] = m;
    }
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (lds_u32(abort_flag)) {
    if (threadIdx.x == 0 && status) atomicOr(status + ENTMAX_ATTN_STATUS_FLAGS, ENTMAX_ATTN_FLAG_WAIT_EXPIRED);
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
    tmem_dealloc(tmem_base, 32);
  }
}

template <int HD>
cudaError_t launch_impl(const DecodeArgs& a, const void* q, const void* k, float* scores, float* chunk_max,
                        int32_t* status, cudaStream_t stream) {
  CUtensorMap map_q, map_k;
  cudaError_t err = make_tile_map(&map_q, q, a.D, a.QL, a.H, a.B, a.D, (int64_t)a.QL * a.D, (int64_t)a.H * a.QL * a.D, kQPad);
  if (err != cudaSuccess) return err;
  err = make_tile_map(&map_k, k, a.D, a.NC, a.H, a.B, a.ksn, a.ksh, a.ksb, kTile);
  if (err != cudaSuccess) return err;
  err = cudaFuncSetAttribute(decode_scores_tc_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, DCfg<HD>::kSmemBytes);
  if (err != cudaSuccess) return err;
  const dim3 grid(a.n_chunks, a.H, a.B);
  decode_scores_tc_kernel<HD><<<grid, kThreadsD, DCfg<HD>::kSmemBytes, stream>>>(map_q, map_k, a, scores, chunk_max,
                                                                                status);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode_scores_tc(const DecodeArgs& a, const void* q, const void* k, float* scores, float* chunk_max,
                                    int32_t* status, cudaStream_t stream) {
  return a.D == 64 ? launch_impl<64>(a, q, k, scores, chunk_max, status, stream)
                   : launch_impl<128>(a, q, k, scores, chunk_max, status, stream);
}

}  // namespace entmax
