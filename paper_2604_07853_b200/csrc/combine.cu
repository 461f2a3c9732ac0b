// Top-k weighted combine: out[t] = bf16( sum_j float(c[t,j]) ), the token's k bf16
// contributions added in ASCENDING EXPERT ID starting from 0.0f -- a fixed order (App. C), so
// the result does not depend on the caller's slot order or on how the batch was tiled.
// contrib is [M*k, H] bf16 indexed by flat pair id, or, with `pos_of_pair`, by the pair's position in
// the expert-sorted order (rows that came back from other GPUs' experts); HBM-bound, 128-bit accesses.
#include "common.cuh"

namespace qarl {
namespace {

constexpr int kMaxTopK = 32;

__global__ void __launch_bounds__(256) combine_kernel(const uint16_t* __restrict__ contrib,
                                                      const int32_t* __restrict__ ids,
                                                      const int32_t* __restrict__ pos_of_pair, int64_t M, int k,
                                                      int64_t H, uint16_t* __restrict__ out, int* status) {
  __shared__ int64_t order[kMaxTopK];  // contrib row of the rank-th smallest expert id of this token
  pdl_trigger();
  pdl_wait();
  const int64_t t = blockIdx.x;
  const int tid = threadIdx.x;
  if (tid < k) {
    const int mine = ids[t * k + tid];
    int rank = 0;
    for (int j = 0; j < k; ++j) {
      const int other = ids[t * k + j];
      if (other < mine || (other == mine && j < tid)) ++rank;
      if (other == mine && j != tid) set_status(status, QARL_ERR_BAD_EXPERT_ID);  // expert repeated in a token
    }
    const int64_t pair = t * k + tid;
    order[rank] = pos_of_pair ? min(max(static_cast<int64_t>(pos_of_pair[pair]), int64_t(0)), M * k - 1) : pair;
  }
  __syncthreads();
  for (int64_t c = static_cast<int64_t>(tid) * 8; c < H; c += 256 * 8) {
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
    for (int a = 0; a < k; ++a) {
      const uint4 v = *reinterpret_cast<const uint4*>(contrib + order[a] * H + c);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        acc[2 * i] = __fadd_rn(acc[2 * i], bf16_bits_to_f32(w[i] & 0xFFFFu));
        acc[2 * i + 1] = __fadd_rn(acc[2 * i + 1], bf16_bits_to_f32(w[i] >> 16));
      }
    }
    uint4 o;
    o.x = pack_bf16x2(acc[0], acc[1]);
    o.y = pack_bf16x2(acc[2], acc[3]);
    o.z = pack_bf16x2(acc[4], acc[5]);
    o.w = pack_bf16x2(acc[6], acc[7]);
    *reinterpret_cast<uint4*>(out + t * H + c) = o;
  }
}

}  // namespace

cudaError_t launch_combine(const Launch& L, const uint16_t* contrib, const int32_t* ids, int64_t M, int64_t k,
                           int64_t H, int64_t E, uint16_t* out, const int32_t* pos_of_pair) {
  (void)E;
  if (M == 0) return cudaSuccess;
  ++*L.launches;
  return launch_pdl(combine_kernel, static_cast<unsigned>(M), 256, 0, L.stream, contrib, ids, pos_of_pair, M,
                    static_cast<int>(k), H, out, L.d_status);
}

}  // namespace qarl
