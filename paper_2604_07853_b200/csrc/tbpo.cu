// TBPO sequence-level surrogate (Sec. 3.2; ratio and weight as written out in the appendix
// "Detail of TBPO") over B packed responses: for response i with tokens [off[i], off[i+1]) of the
// flat fp32 arrays,
//   a = mean_t (lp_cur - lp_old_learner),  r = exp(a);   b = mean_t (lp_old_learner - lp_old_sampler),  w = exp(b)
//   w~ = exp(clip(b, -log c, log c));  r~ = clip(r, 0, 1 + eps_h) if A >= 0 else clip(r, 1 - delta_l, 1 + delta_h)
//   J = w~ r~ A;   loss = -mean_i J;   d loss / d lp_cur[t] = -(w~ A r) / (L B) if r is inside its band, else 0.
// HBM-bound: 12 bytes read and 4 written per token.  The token axis is cut into fixed chunks
// of 8192 tokens so that the work is balanced whatever the response lengths are:
//   map      (thread per response)  first[k] = the response that holds token 8192 k; empty responses are finished here
//   partial  (CTA per chunk)        for every response that overlaps the chunk, the sums of the two token
//                                   differences over the overlap, in double, to slot (response + chunk)
//                                   -- unique, because both indices only grow along the token axis
//   stats    (thread per response)  add the response's partials in chunk order, form r, w, J, flags and the
//                                   gradient value its tokens share, in double; the last CTA to finish adds
//                                   all J in index order: loss = -mean J
//   grad     (CTA per chunk)        streams the per-response gradient value over the response's tokens
// Every sum has a fixed order: results do not depend on the grid or on timing.
#include <math.h>

#include "common.cuh"

namespace qarl {
namespace {

constexpr int kChunk = 8192;
constexpr int kSub = 2048;  // tokens per pass of a CTA: 8 per thread, loads issued together
constexpr int kThreads = 256;

struct TbpoParams {
  const float* lp_cur;
  const float* lp_old;
  const float* lp_smp;
  const int64_t* off;
  const float* adv;
  int64_t B, T;
  double eps_h, delta_l, delta_h, log_cap;
  double* r_seq;
  double* w_seq;
  double* j_seq;
  int32_t* flags;
  float* grad;
  double* loss;
  int32_t* first;    // [nchunks]
  double2* partial;  // [B + nchunks]
  float* gval;       // [B] gradient value shared by the response's tokens
  unsigned int* ticket;  // CTAs of the stats kernel that have finished
};

__device__ __forceinline__ int64_t clamp_off(const TbpoParams& p, int64_t i) {
  return min(max(p.off[i], int64_t(0)), p.T);
}

__global__ void __launch_bounds__(kThreads) tbpo_map_kernel(const TbpoParams p) {
  pdl_trigger();
  pdl_wait();
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i == 0) *p.ticket = 0;
  if (i >= p.B) return;
  const int64_t t0 = clamp_off(p, i), t1 = clamp_off(p, i + 1);
  if (t1 <= t0) {  // empty response: J = 0, still counted in B
    p.r_seq[i] = 1.0;
    p.w_seq[i] = 1.0;
    p.j_seq[i] = 0.0;
    p.flags[i] = 4;
    p.gval[i] = 0.0f;
    return;
  }
  for (int64_t k = (t0 + kChunk - 1) / kChunk; k * kChunk < t1; ++k) p.first[k] = static_cast<int32_t>(i);
}

// Sum of v over the CTA, returned to every thread.  Fixed order: lanes by xor-shuffle, warps in index order.
__device__ __forceinline__ double2 block_sum(double2 v, double2* warp_part) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    v.x += __shfl_xor_sync(0xFFFFFFFFu, v.x, o);
    v.y += __shfl_xor_sync(0xFFFFFFFFu, v.y, o);
  }
  __syncthreads();  // the previous use of warp_part is over
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = v;
  __syncthreads();
  double2 s = warp_part[0];
#pragma unroll
  for (int i = 1; i < kThreads / 32; ++i) {
    s.x += warp_part[i].x;
    s.y += warp_part[i].y;
  }
  return s;
}

__global__ void __launch_bounds__(kThreads) tbpo_partial_kernel(const TbpoParams p) {
  __shared__ double2 warp_part[kThreads / 32];
  pdl_trigger();
  pdl_wait();
  const int64_t k = blockIdx.x;
  const int64_t lo = k * kChunk, hi = min(lo + kChunk, p.T);
  // first[k] is only defined for well-formed offsets (monotone, covering [0, T)); clamped so that
  // malformed ones give wrong numbers, never an out-of-range access
  for (int64_t i = min(max(static_cast<int64_t>(p.first[k]), int64_t(0)), p.B - 1); i < p.B; ++i) {
    const int64_t t0 = clamp_off(p, i);
    if (t0 >= hi) break;
    const int64_t s0 = max(t0, lo), s1 = min(clamp_off(p, i + 1), hi);
    double2 acc = make_double2(0.0, 0.0);
    for (int64_t base = s0; base < s1; base += kSub) {
      float c[8], o[8], q[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int64_t t = base + threadIdx.x + u * kThreads;
        const bool in = t < s1;
        c[u] = in ? __ldg(p.lp_cur + t) : 0.0f;
        o[u] = in ? __ldg(p.lp_old + t) : 0.0f;
        q[u] = in ? __ldg(p.lp_smp + t) : 0.0f;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {  // differences formed in double: exact
        acc.x += static_cast<double>(c[u]) - static_cast<double>(o[u]);
        acc.y += static_cast<double>(o[u]) - static_cast<double>(q[u]);
      }
    }
    const double2 s = block_sum(acc, warp_part);
    if (threadIdx.x == 0 && s1 > s0) p.partial[i + k] = s;
  }
}

__global__ void __launch_bounds__(kThreads) tbpo_stats_kernel(const TbpoParams p) {
  __shared__ double part[kThreads];
  __shared__ bool last;
  pdl_trigger();
  pdl_wait();
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < p.B) {
    const int64_t t0 = clamp_off(p, i), t1 = clamp_off(p, i + 1);
    if (t1 > t0) {
      double sa = 0.0, sb = 0.0;
      for (int64_t kk = t0 / kChunk; kk * kChunk < t1; ++kk) {  // the response's partials in chunk order
        const double2 v = p.partial[i + kk];
        sa += v.x;
        sb += v.y;
      }
      const double L = static_cast<double>(t1 - t0);
      const double a = sa / L, b = sb / L;
      const double r = exp(a);
      int f = 0;
      double bc = b;
      if (bc > p.log_cap) { bc = p.log_cap; f |= 2; }
      if (bc < -p.log_cap) { bc = -p.log_cap; f |= 2; }
      const double wt = exp(bc);
      const double A = static_cast<double>(__ldg(p.adv + i));
      const double band_lo = A >= 0.0 ? 0.0 : 1.0 - p.delta_l;
      const double band_hi = A >= 0.0 ? 1.0 + p.eps_h : 1.0 + p.delta_h;
      double rt = r;
      if (rt < band_lo) { rt = band_lo; f |= 1; }
      if (rt > band_hi) { rt = band_hi; f |= 1; }
      p.r_seq[i] = r;
      p.w_seq[i] = (f & 2) ? exp(b) : wt;
      p.j_seq[i] = wt * rt * A;
      p.flags[i] = f;
      p.gval[i] = (f & 1) ? 0.0f : static_cast<float>(-(wt * A * r) / (L * static_cast<double>(p.B)));
    }
  }
  // The last CTA to get here adds every J in one fixed order (thread j takes j, j + 256, ...; then a
  // tree): which CTA that is varies, what it computes does not.
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last = atomicAdd(p.ticket, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!last) return;
  __threadfence();
  double s = 0.0;
  for (int64_t j = threadIdx.x; j < p.B; j += kThreads) s += __ldcg(p.j_seq + j);
  part[threadIdx.x] = s;
  __syncthreads();
  for (int o = kThreads / 2; o > 0; o >>= 1) {
    if (threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *p.loss = -part[0] / static_cast<double>(p.B);
}

__global__ void __launch_bounds__(kThreads) tbpo_grad_kernel(const TbpoParams p) {
  pdl_trigger();
  pdl_wait();
  const int64_t k = blockIdx.x;
  const int64_t lo = k * kChunk, hi = min(lo + kChunk, p.T);
  for (int64_t i = min(max(static_cast<int64_t>(p.first[k]), int64_t(0)), p.B - 1); i < p.B; ++i) {
    const int64_t t0 = clamp_off(p, i);
    if (t0 >= hi) break;
    const int64_t s0 = max(t0, lo), s1 = min(clamp_off(p, i + 1), hi);
    if (s1 <= s0) continue;
    const float g = __ldg(p.gval + i);
    for (int64_t t = s0 + threadIdx.x; t < s1; t += kThreads) p.grad[t] = g;
  }
}

__global__ void tbpo_zero_loss_kernel(const TbpoParams p) {
  pdl_trigger();
  pdl_wait();
  *p.loss = 0.0;
}

}  // namespace

namespace {
struct TbpoWs {
  size_t first, partial, gval, ticket, total;
};
TbpoWs tbpo_plan(int64_t B, int64_t T) {
  const int64_t nchunks = (T + kChunk - 1) / kChunk;
  auto up = [](size_t v) { return (v + 255) / 256 * 256; };
  TbpoWs w{};
  w.first = 0;
  w.partial = up(static_cast<size_t>(nchunks) * sizeof(int32_t));
  w.gval = w.partial + up(static_cast<size_t>(B + nchunks) * sizeof(double2));
  w.ticket = w.gval + up(static_cast<size_t>(B) * sizeof(float));
  w.total = w.ticket + 256;
  return w;
}
}  // namespace

size_t tbpo_workspace_bytes(int64_t B, int64_t T) { return tbpo_plan(B, T).total; }

cudaError_t launch_tbpo(const Launch& L, const TbpoArgs& a) {
  TbpoParams p{};
  p.lp_cur = a.lp_cur;
  p.lp_old = a.lp_old_learner;
  p.lp_smp = a.lp_old_sampler;
  p.off = a.offsets;
  p.adv = a.adv;
  p.B = a.B;
  p.T = a.T;
  p.eps_h = a.eps_h;
  p.delta_l = a.delta_l;
  p.delta_h = a.delta_h;
  p.log_cap = log(a.cap);
  p.r_seq = a.r_seq;
  p.w_seq = a.w_seq;
  p.j_seq = a.j_seq;
  p.flags = a.flags;
  p.grad = a.grad;
  p.loss = a.loss;
  const int64_t nchunks = (a.T + kChunk - 1) / kChunk;
  const TbpoWs w = tbpo_plan(a.B, a.T);
  uint8_t* ws = static_cast<uint8_t*>(a.workspace);
  p.first = reinterpret_cast<int32_t*>(ws + w.first);
  p.partial = reinterpret_cast<double2*>(ws + w.partial);
  p.gval = reinterpret_cast<float*>(ws + w.gval);
  p.ticket = reinterpret_cast<unsigned int*>(ws + w.ticket);
  if (a.B == 0) {  // no responses: the loss of an empty batch is 0
    ++*L.launches;
    return launch_pdl(tbpo_zero_loss_kernel, 1u, 1u, 0, L.stream, p);
  }
  const unsigned resp_blocks = static_cast<unsigned>((a.B + kThreads - 1) / kThreads);
  ++*L.launches;
  cudaError_t e = launch_pdl(tbpo_map_kernel, resp_blocks, kThreads, 0, L.stream, p);
  if (e != cudaSuccess) return e;
  if (nchunks > 0) {
    ++*L.launches;
    e = launch_pdl(tbpo_partial_kernel, static_cast<unsigned>(nchunks), kThreads, 0, L.stream, p);
    if (e != cudaSuccess) return e;
  }
  ++*L.launches;
  e = launch_pdl(tbpo_stats_kernel, resp_blocks, kThreads, 0, L.stream, p);
  if (e != cudaSuccess) return e;
  if (nchunks > 0 && a.grad) {
    ++*L.launches;
    e = launch_pdl(tbpo_grad_kernel, static_cast<unsigned>(nchunks), kThreads, 0, L.stream, p);
  }
  return e;
}

}  // namespace qarl
