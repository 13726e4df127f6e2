// Declarations shared by the decode-shape kernels (decode.cu, decode_scores_sm100.cu).
#pragma once

#include "common.cuh"

namespace entmax {

struct DecodeArgs {
  int B, H, QL, NC, D;             // NC = kv_capacity
  int expo_class;
  float expo, alpha_m1, sm_scale;
  int64_t ksb, ksh, ksn;           // element strides of K and V
  const int32_t* kv_len;           // [B] or nullptr
  const float* alibi;              // [H] or nullptr
  const float *beta, *gamma, *delta;   // [H] each, or all nullptr (c = 1)
  int chunk_keys;                  // keys per chunk maximum (a multiple of 128)
  int n_chunks;
  size_t score_stride;             // floats per score row
};

__device__ __forceinline__ int seq_len(const DecodeArgs& a, int b, int32_t* status) {
  int len = a.kv_len ? a.kv_len[b] : a.NC;
  if (len < a.QL || len > a.NC) {
    if (status) atomicOr(status + ENTMAX_ATTN_STATUS_FLAGS, ENTMAX_ATTN_FLAG_BAD_LENGTH);
    len = len < a.QL ? a.QL : a.NC;
  }
  return len;
}

// Score stream on the tensor cores: K tiles of 128 keys as the M side of tcgen05 MMAs against the (zero-padded)
// query rows, one thread per key afterwards.  Writes the score rows and the chunk maxima.
cudaError_t launch_decode_scores_tc(const DecodeArgs& a, const void* q, const void* k, float* scores, float* chunk_max,
                                    int32_t* status, cudaStream_t stream);

}  // namespace entmax
