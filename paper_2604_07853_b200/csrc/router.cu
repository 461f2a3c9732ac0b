// Router of the MoE block: top-k experts of every token from its fp32 logits (ties to the lower
// expert id, descending order) and the softmax over the selected logits.  One warp per token; lane l
// keeps experts l, l + 32, ... in registers; k rounds of a warp arg-max.  The logits come from the
// bf16 tensor-core GEMM (x . W_r^T, fp32 accumulation in a fixed order), so a token's routing
// depends only on that token's row -- the same invariance the expert GEMMs have (App. C).
#include <math.h>

#include "common.cuh"

namespace qarl {
namespace {

// PER = experts per lane (E <= 32 PER), a compile-time bound so that the selection loops unroll to
// exactly the work the expert count needs.
template <int PER>
__global__ void __launch_bounds__(256) router_topk_kernel(const float* __restrict__ logits, int64_t M, int E, int k,
                                                          int32_t* __restrict__ ids, float* __restrict__ wts) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t m = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  if (m >= M) return;
  const float* row = logits + m * E;
  float v[PER];
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int e = lane + 32 * j;
    v[j] = e < E ? row[e] : -INFINITY;
  }
  uint32_t taken = 0;  // bit j: this lane's j-th expert was selected
  float sel = 0.0f;    // lane j < k ends up holding the j-th selected logit
  int sel_id = 0;
  for (int r = 0; r < k; ++r) {
    float best = -INFINITY;
    int best_e = 0x7FFFFFFF;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (!((taken >> j) & 1u)) {
        const int e = lane + 32 * j;
        if (e < E && (v[j] > best || best_e == 0x7FFFFFFF)) {  // ascending e within a lane: strict > keeps the lower id
          best = v[j];
          best_e = e;
        }
      }
    }
    // Warp arg-max in two reductions instead of a five-step butterfly on (value, id) pairs: the largest
    // value through an order-preserving map of its bits to unsigned (-0 first folded onto +0, so equal
    // values map to equal keys), then the lowest id among the lanes that hold it.
    const uint32_t bits = __float_as_uint(best + 0.0f);
    const uint32_t key = best_e == 0x7FFFFFFF ? 0u : ((bits & 0x80000000u) ? ~bits : (bits | 0x80000000u));
    const uint32_t top = __reduce_max_sync(0xFFFFFFFFu, key);
    const int win_e = static_cast<int>(__reduce_min_sync(0xFFFFFFFFu, key == top ? static_cast<uint32_t>(best_e) : 0x7FFFFFFFu));
    const float win = __shfl_sync(0xFFFFFFFFu, best, win_e & 31);
    best = win;
    best_e = win_e;
    if ((best_e & 31) == lane) taken |= 1u << (best_e >> 5);
    if (lane == r) {
      sel = best;
      sel_id = best_e;
    }
  }
  // softmax over the k selected logits, in double: exp(l - max) / sum, rounded to fp32
  const double mx = static_cast<double>(__shfl_sync(0xFFFFFFFFu, sel, 0));
  double ex = lane < k ? exp(static_cast<double>(sel) - mx) : 0.0;
  double den = 0.0;  // summed in selection order (the one-launch router adds them as it selects)
  for (int j = 0; j < k; ++j) den += __shfl_sync(0xFFFFFFFFu, ex, j);
  if (lane < k) {
    ids[m * k + lane] = sel_id;
    wts[m * k + lane] = static_cast<float>(ex / den);
  }
}

}  // namespace

cudaError_t launch_router_topk(const Launch& L, const float* logits, int64_t M, int64_t E, int64_t k, int32_t* ids,
                               float* wts) {
  if (M == 0) return cudaSuccess;
  ++*L.launches;
  const unsigned grid = static_cast<unsigned>((M * 32 + 255) / 256);
  const int Ei = static_cast<int>(E), ki = static_cast<int>(k);
  const int per = static_cast<int>((E + 31) / 32);
  if (per <= 1) return launch_pdl(router_topk_kernel<1>, grid, 256, 0, L.stream, logits, M, Ei, ki, ids, wts);
  if (per <= 2) return launch_pdl(router_topk_kernel<2>, grid, 256, 0, L.stream, logits, M, Ei, ki, ids, wts);
  if (per <= 4) return launch_pdl(router_topk_kernel<4>, grid, 256, 0, L.stream, logits, M, Ei, ki, ids, wts);
  if (per <= 8) return launch_pdl(router_topk_kernel<8>, grid, 256, 0, L.stream, logits, M, Ei, ki, ids, wts);
  if (per <= 16) return launch_pdl(router_topk_kernel<16>, grid, 256, 0, L.stream, logits, M, Ei, ki, ids, wts);
  return launch_pdl(router_topk_kernel<32>, grid, 256, 0, L.stream, logits, M, Ei, ki, ids, wts);
}

}  // namespace qarl
