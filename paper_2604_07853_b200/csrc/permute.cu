// Token-expert grouping: a stable counting sort of the M*k flat pairs p = t*k + j by expert
// id, built from warp-level match/ballot prefix sums.  Output (exactly one correct answer):
//   offsets[e]     first sorted position of expert e, offsets[E] = P
//   sorted_pair[q] the pair at sorted position q (ties by ascending pair id)
//   pos_of_pair[p] the inverse permutation
// Integer work only.  Ids outside [0, E) are reported through the status word and skipped
// (nothing is written for them), so the kernels stay memory-safe on bad input.
#include <algorithm>

#include "common.cuh"
#include "quant_device.cuh"

namespace qarl {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kPairsPerWarp = 256;
constexpr int kChunk = kWarps * kPairsPerWarp;  // 2048 pairs per CTA

// Lanes of the warp whose id equals this lane's id (what match.any gives), from one ballot per id
// bit: ten ballots cover every id below 1024 and -1 (a bad id, all ones in the low bits too: it is
// told apart by the eleventh ballot).  match.any itself measured about a microsecond per call here,
// which made the grouping the slowest kernel of a decode step.
__device__ __forceinline__ uint32_t match_id(int e) {
  uint32_t peers = 0xFFFFFFFFu;
#pragma unroll
  for (int b = 0; b < 11; ++b) {
    const uint32_t bit = (static_cast<uint32_t>(e) >> (b == 10 ? 31 : b)) & 1u;
    const uint32_t v = __ballot_sync(0xFFFFFFFFu, bit);
    peers &= bit ? v : ~v;
  }
  return peers;
}

// Per-warp histogram of the warp's contiguous 256-pair slice into hist_w[0..E).  Lanes with
// equal ids are found with match_any; the lowest such lane adds the group's size, so no
// atomics are needed (one warp owns hist_w).
__device__ __forceinline__ void warp_histogram(const int32_t* __restrict__ ids, int64_t p0, int64_t P, int E,
                                               int32_t* hist_w, int* status) {
  const int lane = threadIdx.x & 31;
  for (int r = 0; r < kPairsPerWarp / 32; ++r) {
    const int64_t p = p0 + r * 32 + lane;
    int e = -1;
    if (p < P) {
      e = ids[p];
      if (e < 0 || e >= E) {
        set_status(status, QARL_ERR_BAD_EXPERT_ID);
        e = -1;
      }
    }
    const uint32_t peers = match_id(e);
    if (e >= 0 && (__ffs(peers) - 1) == lane) hist_w[e] += __popc(peers);
    __syncwarp();
  }
}

// Walk the warp's slice again in order; cursor_w[e] holds the next free sorted position for
// expert e within this warp's slice.  rank among equal-id lanes = popc(peers below me).
__device__ __forceinline__ void warp_scatter(const int32_t* __restrict__ ids, int64_t p0, int64_t P, int E,
                                             int32_t* cursor_w, int32_t* __restrict__ sorted_pair,
                                             int32_t* __restrict__ pos_of_pair) {
  const int lane = threadIdx.x & 31;
  const uint32_t lt = (1u << lane) - 1u;
  for (int r = 0; r < kPairsPerWarp / 32; ++r) {
    const int64_t p = p0 + r * 32 + lane;
    int e = -1;
    if (p < P) {
      e = ids[p];
      if (e < 0 || e >= E) e = -1;
    }
    const uint32_t peers = match_id(e);
    int pos = -1;
    if (e >= 0) pos = cursor_w[e] + __popc(peers & lt);
    __syncwarp();
    if (e >= 0 && (__ffs(peers) - 1) == lane) cursor_w[e] += __popc(peers);
    __syncwarp();
    if (e >= 0) {
      sorted_pair[pos] = static_cast<int32_t>(p);
      pos_of_pair[p] = pos;
    }
  }
}

// Exclusive scan of a[0..n) in shared memory by the whole CTA (n <= 1024); returns the total.
// scratch: 33 ints of shared memory.
__device__ int block_exclusive_scan(int32_t* a, int n, int32_t* scratch) {
  const int tid = threadIdx.x, nt = blockDim.x;
  const int items = (n + nt - 1) / nt;
  const int i0 = tid * items;
  int sum = 0;
  for (int i = 0; i < items; ++i)
    if (i0 + i < n) sum += a[i0 + i];
  // inclusive warp scan of the per-thread sums
  int inc = sum;
  const int lane = tid & 31, wid = tid >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xFFFFFFFFu, inc, o);
    if (lane >= o) inc += v;
  }
  if (lane == 31) scratch[wid] = inc;
  __syncthreads();
  if (wid == 0) {
    const int nw = nt >> 5;
    int v = lane < nw ? scratch[lane] : 0;
    int vi = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xFFFFFFFFu, vi, o);
      if (lane >= o) vi += u;
    }
    if (lane < nw) scratch[lane] = vi - v;  // exclusive warp bases
    if (lane == 31) scratch[32] = vi;       // total
  }
  __syncthreads();
  int run = scratch[wid] + inc - sum;
  for (int i = 0; i < items; ++i)
    if (i0 + i < n) {
      const int v = a[i0 + i];
      a[i0 + i] = run;
      run += v;
    }
  __syncthreads();
  return scratch[32];
}

// ---- small problems (P <= 2048): one CTA does histogram, scan and scatter ----------------
// Each lane keeps its 8 ids in registers for both passes, so global memory is read once and
// the eight loads are in flight together (this kernel is pure latency at decode sizes).
__global__ void __launch_bounds__(kThreads) permute_single_cta_kernel(const int32_t* __restrict__ ids, int64_t P,
                                                                      int E, int32_t* __restrict__ offsets,
                                                                      int32_t* __restrict__ sorted_pair,
                                                                      int32_t* __restrict__ pos_of_pair,
                                                                      int* status) {
  extern __shared__ int32_t sm[];
  pdl_trigger();
  pdl_wait();
  int32_t* whist = sm;                 // [kWarps][E]
  int32_t* total = sm + kWarps * E;    // [E]
  int32_t* scratch = total + E;        // [33]
  const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
  constexpr int kRounds = kPairsPerWarp / 32;
  const int64_t p0 = static_cast<int64_t>(wid) * kPairsPerWarp + lane;
  int my[kRounds];
  bool bad = false;
#pragma unroll
  for (int r = 0; r < kRounds; ++r) {
    const int64_t p = p0 + r * 32;
    int e = -1;
    if (p < P) {
      e = __ldg(ids + p);
      if (e < 0 || e >= E) { bad = true; e = -1; }
    }
    my[r] = e;
  }
  if (bad) set_status(status, QARL_ERR_BAD_EXPERT_ID);
  for (int i = tid; i < kWarps * E; i += kThreads) whist[i] = 0;
  __syncthreads();
  int32_t* hist_w = whist + wid * E;
#pragma unroll
  for (int r = 0; r < kRounds; ++r) {
    const int e = my[r];
    const uint32_t peers = match_id(e);
    if (e >= 0 && (__ffs(peers) - 1) == lane) hist_w[e] += __popc(peers);
    __syncwarp();
  }
  __syncthreads();
  for (int e = tid; e < E; e += kThreads) {
    int s = 0;
    for (int w = 0; w < kWarps; ++w) s += whist[w * E + e];
    total[e] = s;
  }
  __syncthreads();
  const int all = block_exclusive_scan(total, E, scratch);
  for (int e = tid; e < E; e += kThreads) {
    int run = total[e];
    offsets[e] = run;
    for (int w = 0; w < kWarps; ++w) {
      const int c = whist[w * E + e];
      whist[w * E + e] = run;
      run += c;
    }
  }
  if (tid == 0) offsets[E] = all;
  __syncthreads();
  const uint32_t lt = (1u << lane) - 1u;
#pragma unroll
  for (int r = 0; r < kRounds; ++r) {
    const int e = my[r];
    const uint32_t peers = match_id(e);
    int pos = -1;
    if (e >= 0) pos = hist_w[e] + __popc(peers & lt);
    __syncwarp();
    if (e >= 0 && (__ffs(peers) - 1) == lane) hist_w[e] += __popc(peers);
    __syncwarp();
    if (e >= 0) {
      const int64_t p = p0 + r * 32;
      sorted_pair[pos] = static_cast<int32_t>(p);
      pos_of_pair[p] = pos;
    }
  }
}

// ---- decode-sized layers (P <= 2048): grouping + activation quantization in ONE launch --------
// Every CTA repeats the whole (tiny, deterministic) grouping in its shared memory -- the ids are 8 KB
// and sit in L2 -- and then quantizes its own share of the activation groups, writing each token's
// codes, scales and combine weight to the token's k expert-sorted rows.  CTA 0 also publishes offsets,
// sorted_pair and pos_of_pair.  One launch and one dependency instead of two of each; the loads of
// the activations are issued before the grouping so that their latency hides behind it.
// 16 warps of 128 pairs: four rounds per pass (the grouping is a chain of short dependent steps, so
// more, shorter warps finish it sooner)
constexpr int kPrepThreads = 512;
constexpr int kPrepWarps = kPrepThreads / 32;
constexpr int kPrepPairsPerWarp = kChunk / kPrepWarps;
__global__ void __launch_bounds__(kPrepThreads) moe_prep_small_kernel(
    const int32_t* __restrict__ ids, int64_t P, int E, int fanout, const uint16_t* __restrict__ x, int64_t M, int64_t K,
    const float* __restrict__ pair_w, int32_t* __restrict__ offsets, int32_t* __restrict__ sorted_pair,
    int32_t* __restrict__ pos_of_pair, uint8_t* __restrict__ codes, float* __restrict__ scales,
    float* __restrict__ sorted_w, int32_t* __restrict__ zero, int zero_count, int* status) {
  extern __shared__ int32_t sm[];
  pdl_trigger();
  pdl_wait();
  if (blockIdx.x == 0)
    for (int i = threadIdx.x; i < zero_count; i += kPrepThreads) zero[i] = 0;
  int32_t* whist = sm;                 // [kPrepWarps][E]
  int32_t* total = sm + kPrepWarps * E;    // [E]
  int32_t* scratch = total + E;        // [33]
  int32_t* spos = scratch + 33;        // [kChunk] sorted position of every pair (-1: bad id)
  const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
  const bool publish = blockIdx.x == 0;

  // this thread's share of the quantization: 16 elements of one 1x128 group
  const int64_t kb = K / kBlock;
  const int64_t gid = (static_cast<int64_t>(blockIdx.x) * blockDim.x + tid) >> 3;
  const bool live = gid < M * kb;
  const int64_t g = live ? gid : 0;
  const int64_t row = g / kb, b = g % kb;
  const int sub = tid & 7;
  uint4 v0 = make_uint4(0, 0, 0, 0), v1 = v0;
  if (live) {
    const uint4* src = reinterpret_cast<const uint4*>(x + row * K + b * kBlock + sub * 16);
    v0 = __ldg(src);
    v1 = __ldg(src + 1);
  }

  // ---- the grouping (as permute_single_cta_kernel), positions kept in shared memory
  constexpr int kRounds = kPrepPairsPerWarp / 32;
  const int64_t p0 = static_cast<int64_t>(wid) * kPrepPairsPerWarp + lane;
  int my[kRounds];
  bool bad = false;
#pragma unroll
  for (int r = 0; r < kRounds; ++r) {
    const int64_t p = p0 + r * 32;
    int e = -1;
    if (p < P) {
      e = __ldg(ids + p);
      if (e < 0 || e >= E) { bad = true; e = -1; }
    }
    my[r] = e;
  }
  if (bad && publish) set_status(status, QARL_ERR_BAD_EXPERT_ID);
  for (int i = tid; i < kPrepWarps * E; i += kPrepThreads) whist[i] = 0;
  for (int i = tid; i < kChunk; i += kPrepThreads) spos[i] = -1;
  __syncthreads();
  int32_t* hist_w = whist + wid * E;
#pragma unroll
  for (int r = 0; r < kRounds; ++r) {
    const int e = my[r];
    const uint32_t peers = match_id(e);
    if (e >= 0 && (__ffs(peers) - 1) == lane) hist_w[e] += __popc(peers);
    __syncwarp();
  }
  __syncthreads();
  for (int e = tid; e < E; e += kPrepThreads) {
    int s = 0;
    for (int w = 0; w < kPrepWarps; ++w) s += whist[w * E + e];
    total[e] = s;
  }
  __syncthreads();
  const int all = block_exclusive_scan(total, E, scratch);
  for (int e = tid; e < E; e += kPrepThreads) {
    int run = total[e];
    if (publish) offsets[e] = run;
    for (int w = 0; w < kPrepWarps; ++w) {
      const int c = whist[w * E + e];
      whist[w * E + e] = run;
      run += c;
    }
  }
  if (publish && tid == 0) offsets[E] = all;
  __syncthreads();
  const uint32_t lt = (1u << lane) - 1u;
#pragma unroll
  for (int r = 0; r < kRounds; ++r) {
    const int e = my[r];
    const uint32_t peers = match_id(e);
    int pos = -1;
    if (e >= 0) pos = hist_w[e] + __popc(peers & lt);
    __syncwarp();
    if (e >= 0 && (__ffs(peers) - 1) == lane) hist_w[e] += __popc(peers);
    __syncwarp();
    if (e >= 0) {
      const int64_t p = p0 + r * 32;
      spos[p] = pos;
      if (publish) {
        sorted_pair[pos] = static_cast<int32_t>(p);
        pos_of_pair[p] = pos;
      }
    }
  }
  __syncthreads();

  // ---- quantize this thread's group and scatter it to the token's sorted rows
  uint32_t m = fold_halves(absmax_u4(absmax_u4(0, v0), v1));
#pragma unroll
  for (int o = 4; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  float inv;
  const float s = block_scale(bf16_bits_to_f32(m), &inv);
  uint4 out;
  encode8(v0, inv, out.x, out.y);
  encode8(v1, inv, out.z, out.w);
  if (!live) return;
  for (int j = 0; j < fanout; ++j) {
    const int d = spos[row * fanout + j];
    if (d < 0) continue;  // a pair with a bad expert id has no sorted row
    *reinterpret_cast<uint4*>(codes + static_cast<int64_t>(d) * K + b * kBlock + sub * 16) = out;
    if (sub == 0) scales[static_cast<int64_t>(d) * kb + b] = s;
    if (sub == 0 && b == 0 && sorted_w != nullptr) sorted_w[d] = pair_w[row * fanout + j];
  }
}

// ---- large problems: per-chunk histogram, one-CTA scan, per-chunk scatter ----------------
__global__ void __launch_bounds__(kThreads) permute_hist_kernel(const int32_t* __restrict__ ids, int64_t P, int E,
                                                                int32_t* __restrict__ chunk_hist, int* status) {
  extern __shared__ int32_t sm[];
  pdl_trigger();
  pdl_wait();
  int32_t* whist = sm;
  const int tid = threadIdx.x, wid = tid >> 5;
  for (int i = tid; i < kWarps * E; i += kThreads) whist[i] = 0;
  __syncthreads();
  const int64_t p0 = static_cast<int64_t>(blockIdx.x) * kChunk + static_cast<int64_t>(wid) * kPairsPerWarp;
  warp_histogram(ids, p0, P, E, whist + wid * E, status);
  __syncthreads();
  for (int e = tid; e < E; e += kThreads) {
    int s = 0;
    for (int w = 0; w < kWarps; ++w) s += whist[w * E + e];
    chunk_hist[static_cast<int64_t>(blockIdx.x) * E + e] = s;
  }
}

// One CTA of 1024 threads.  Turns chunk_hist[c][e] into the exclusive running count of expert
// e over chunks 0..c-1 and writes the expert offsets.  Threads are laid out (g, e): group g
// handles a contiguous range of chunks for expert e so the chunk walk is G-way parallel.
__global__ void __launch_bounds__(1024) permute_scan_kernel(int32_t* __restrict__ chunk_hist, int nchunks, int E,
                                                            int32_t* __restrict__ offsets) {
  extern __shared__ int32_t sm[];
  pdl_trigger();
  pdl_wait();
  const int G = max(1, min(static_cast<int>(blockDim.x) / E, nchunks));
  int32_t* part = sm;            // [G][E]
  int32_t* total = sm + G * E;   // [E]
  int32_t* scratch = total + E;  // [33]
  const int tid = threadIdx.x;
  const int cpg = (nchunks + G - 1) / G;
  const int g = tid / E, e = tid % E;
  const bool active = g < G;
  const int c0 = g * cpg, c1 = min(c0 + cpg, nchunks);
  if (active) {
    int s = 0;
    for (int c = c0; c < c1; ++c) s += chunk_hist[static_cast<int64_t>(c) * E + e];
    part[g * E + e] = s;
  }
  __syncthreads();
  if (tid < E) {
    int run = 0;
    for (int gg = 0; gg < G; ++gg) {
      const int v = part[gg * E + tid];
      part[gg * E + tid] = run;
      run += v;
    }
    total[tid] = run;
  }
  __syncthreads();
  const int all = block_exclusive_scan(total, E, scratch);
  if (tid < E) offsets[tid] = total[tid];
  if (tid == 0) offsets[E] = all;
  if (active) {
    int run = part[g * E + e];
    for (int c = c0; c < c1; ++c) {
      const int64_t i = static_cast<int64_t>(c) * E + e;
      const int v = chunk_hist[i];
      chunk_hist[i] = run;
      run += v;
    }
  }
}

__global__ void __launch_bounds__(kThreads) permute_scatter_kernel(const int32_t* __restrict__ ids, int64_t P, int E,
                                                                   const int32_t* __restrict__ chunk_hist,
                                                                   const int32_t* __restrict__ offsets,
                                                                   int32_t* __restrict__ sorted_pair,
                                                                   int32_t* __restrict__ pos_of_pair, int* status) {
  extern __shared__ int32_t sm[];
  pdl_trigger();
  pdl_wait();
  int32_t* whist = sm;
  const int tid = threadIdx.x, wid = tid >> 5;
  for (int i = tid; i < kWarps * E; i += kThreads) whist[i] = 0;
  __syncthreads();
  const int64_t p0 = static_cast<int64_t>(blockIdx.x) * kChunk + static_cast<int64_t>(wid) * kPairsPerWarp;
  warp_histogram(ids, p0, P, E, whist + wid * E, status);
  __syncthreads();
  for (int e = tid; e < E; e += kThreads) {
    int run = offsets[e] + chunk_hist[static_cast<int64_t>(blockIdx.x) * E + e];
    for (int w = 0; w < kWarps; ++w) {
      const int c = whist[w * E + e];
      whist[w * E + e] = run;
      run += c;
    }
  }
  __syncthreads();
  warp_scatter(ids, p0, P, E, whist + wid * E, sorted_pair, pos_of_pair);
}

}  // namespace

int64_t permute_num_chunks(int64_t P) { return (P + kChunk - 1) / kChunk; }

bool moe_prep_small_applies(int64_t M, int64_t k, int64_t E) { return M * k <= kChunk && E <= 1024; }

cudaError_t launch_moe_prep_small(const Launch& L, const int32_t* ids, int64_t M, int64_t k, int64_t E,
                                  const PermuteBuffers& b, const uint16_t* x, int64_t K, const float* pair_w,
                                  uint8_t* codes, float* scales, float* sorted_w, int32_t* zero, int zero_count) {
  const int e = static_cast<int>(E);
  const size_t smem = (static_cast<size_t>(kPrepWarps) * e + e + 33 + kChunk) * sizeof(int32_t);
  if (smem > 48 * 1024) {
    cudaError_t err = cudaFuncSetAttribute(moe_prep_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           static_cast<int>(smem));
    if (err != cudaSuccess) return err;
  }
  const int64_t groups = M * (K / kBlock);
  const int64_t blocks = std::max<int64_t>(1, (groups * 8 + kPrepThreads - 1) / kPrepThreads);
  ++*L.launches;
  return launch_pdl(moe_prep_small_kernel, static_cast<unsigned>(blocks), kPrepThreads, smem, L.stream, ids, M * k, e,
                    static_cast<int>(k), x, M, K, pair_w, b.offsets, b.sorted_pair, b.pos_of_pair, codes, scales, sorted_w,
                    zero, zero_count, L.d_status);
}

cudaError_t launch_permute(const Launch& L, const int32_t* ids, int64_t M, int64_t k, int64_t E,
                           const PermuteBuffers& b) {
  const int64_t P = M * k;
  const int e = static_cast<int>(E);
  const int64_t nchunks = permute_num_chunks(P);
  cudaError_t err;
  if (nchunks <= 1) {
    const size_t smem = (static_cast<size_t>(kWarps) * e + e + 33) * sizeof(int32_t);
    if (smem > 48 * 1024) {
      err = cudaFuncSetAttribute(permute_single_cta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem));
      if (err != cudaSuccess) return err;
    }
    ++*L.launches;
    return launch_pdl(permute_single_cta_kernel, 1, kThreads, smem, L.stream, ids, P, e, b.offsets, b.sorted_pair,
                      b.pos_of_pair, L.d_status);
  }
  const size_t smem_h = static_cast<size_t>(kWarps) * e * sizeof(int32_t);
  const int G = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(1024 / e, nchunks)));
  const size_t smem_s = (static_cast<size_t>(G) * e + e + 33) * sizeof(int32_t);
  *L.launches += 3;
  if ((err = launch_pdl(permute_hist_kernel, static_cast<unsigned>(nchunks), kThreads, smem_h, L.stream, ids, P, e,
                        b.chunk_hist, L.d_status)) != cudaSuccess)
    return err;
  if ((err = launch_pdl(permute_scan_kernel, 1, 1024, smem_s, L.stream, b.chunk_hist, static_cast<int>(nchunks), e,
                        b.offsets)) != cudaSuccess)
    return err;
  return launch_pdl(permute_scatter_kernel, static_cast<unsigned>(nchunks), kThreads, smem_h, L.stream, ids, P, e,
                    b.chunk_hist, b.offsets, b.sorted_pair, b.pos_of_pair, L.d_status);
}

}  // namespace qarl
