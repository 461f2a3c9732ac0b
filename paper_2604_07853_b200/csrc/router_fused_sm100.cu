// Router forward in one launch for E <= 128 experts and k <= 16: the logits tile of 128 tokens x E experts is
// accumulated on the tensor cores (bf16 operands, fp32 accumulation in TMEM, ascending k -- the
// same MMA sequence per token row as the two-launch path, so the logits are the same bytes), and
// the epilogue warps, one thread per token, take the row out of TMEM, store the logits, select
// the top-k experts (ties to the lower id, descending order) and write the softmax over the
// selected logits.  The routing decision is part of the forward that the sampler and the learner
// must agree on (Sec. 4.2, "router shift"): a token's ids and weights depend only on its own row.
//
// The kernel is bound by streaming x from HBM once (M x H bf16); the logits never make the round
// trip through memory that a separate selection kernel needs.
//
// Structure of a CTA (192 threads, persistent, static schedule over 128-token tiles):
//   warp 4   TMA producer: per 64-element contraction step one box of x (128 tokens x 128 B) and
//            one box of W_r (128 expert rows x 128 B, rows past E zero-filled) into a 4-deep ring;
//   warp 5   MMA issuer: 4 x tcgen05.mma kind::f16 (128 x 128 x 16) per step into one of two
//            128-column TMEM accumulators;
//   warps 0-3  epilogue: thread r owns token row r of the tile (TMEM lane r): 128 fp32 logits in
//            registers, the accumulator handed back at once; the logits go out through a swizzled
//            shared-memory tile and TMA stores (whole lines, clipped at M and E); then the k rounds
//            of the selection (the best of eight per-group candidates, then a re-scan of the winner's
//            16-expert group) and the softmax in double (exp of logit - max, summed in selection
//            order), while the next tile's main loop runs.
// Every wait is bounded (status word + CTA-wide abort flag), as in the GEMMs.
#include <algorithm>
#include <atomic>
#include <math.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace qarl {
namespace {

using namespace ptx;

constexpr int RM = 128;       // tokens per tile (UMMA M)
constexpr int RN = 128;       // experts per tile (UMMA N)
constexpr int RK = 64;        // contraction elements per stage: one 128-byte swizzle span of bf16
constexpr int kStages = 4;    // measured: 4, 5 and 6 stages run alike; the rest of the shared memory stages the logits
constexpr int kAccBufs = 2;
constexpr int kEpiWarps = 4;  // warps 0-3 (TMEM lane quadrant = warp index)
constexpr int kTmaWarp = 4;
constexpr int kMmaWarp = 5;
constexpr int kThreads = 6 * 32;
constexpr uint32_t kABytes = RM * RK * 2;  // 16 KB
constexpr uint32_t kBBytes = RN * RK * 2;  // 16 KB
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr uint32_t kTmemCols = kAccBufs * RN;
constexpr int kMaxTopK = 16;
constexpr uint32_t kScratchBytes = kMaxTopK * RM * sizeof(double);  // exp values of a row's selection, [round][thread]
// logits of a tile on their way out: per epilogue warp RN / 32 boxes of 32 rows x 128 bytes (128-byte swizzle)
constexpr uint32_t kLogitBoxBytes = 32 * 128;
constexpr uint32_t kLogitBytes = kEpiWarps * (RN / 32) * kLogitBoxBytes;  // 64 KB

struct RouterParams {
  int M, H, E, k;
  float* logits;
  int32_t* ids;
  float* wts;
  int* status;
  unsigned long long wait_limit_ns;
  int stop_after_stages;  // test harness only (< 0: off): the TMA producer stops arming stages after this many
};

struct __align__(8) SmemTail {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t tmem_full[kAccBufs];
  uint64_t tmem_empty[kAccBufs];
  uint64_t teardown;
  uint32_t tmem_addr;
  int abort_flag;
};

constexpr size_t kSmemBytes = 1024 + static_cast<size_t>(kStages) * kStageBytes + kLogitBytes + kScratchBytes + sizeof(SmemTail);
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, SmemTail* s, const RouterParams& p) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 128; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*reinterpret_cast<volatile int*>(&s->abort_flag)) return false;
    if (globaltimer_ns() - t0 > p.wait_limit_ns) {
      set_status(p.status, QARL_ERR_DEVICE_TIMEOUT);
      *reinterpret_cast<volatile int*>(&s->abort_flag) = 1;
      return false;
    }
  }
}

__device__ __forceinline__ bool warp_wait_or_abort(uint64_t* bar, uint32_t parity, SmemTail* s, const RouterParams& p) {
  return __all_sync(0xFFFFFFFFu, wait_or_abort(bar, parity, s, p) ? 1 : 0) != 0;
}

__global__ void __launch_bounds__(kThreads, 1)
router_fused_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                    const __grid_constant__ CUtensorMap tm_l, const RouterParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* logit_tile = smem + static_cast<size_t>(kStages) * kStageBytes;  // 1 KB aligned: the swizzle follows the address
  double* scratch = reinterpret_cast<double*>(logit_tile + kLogitBytes);
  SmemTail* s = reinterpret_cast<SmemTail*>(logit_tile + kLogitBytes + kScratchBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  pdl_trigger();
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&s->full[i], 1);
      mbar_init(&s->empty[i], 1);
    }
    for (int i = 0; i < kAccBufs; ++i) {
      mbar_init(&s->tmem_full[i], 1);
      mbar_init(&s->tmem_empty[i], kEpiWarps);
    }
    mbar_init(&s->teardown, 1);
    s->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kTmaWarp && lane == 0) {
    prefetch_tensormap(&tm_x);
    prefetch_tensormap(&tm_w);
    prefetch_tensormap(&tm_l);
  }
  if (warp == kMmaWarp) {
    tmem_alloc(&s->tmem_addr, kTmemCols);
    tmem_relinquish();
  }
  pdl_wait();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = s->tmem_addr;
  const int total_tiles = (p.M + RM - 1) / RM;
  const int KS = (p.H + RK - 1) / RK;  // a ragged last step reads zeros (TMA out-of-range fill)
  const int grid = gridDim.x;

  if (warp == kTmaWarp) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t armed = 0, armed_parity = 0;
      bool ok = true;
      int armed_total = 0;
      for (int T = blockIdx.x; ok && T < total_tiles; T += grid) {
        for (int ks = 0; ks < KS; ++ks) {
          if (p.stop_after_stages >= 0 && armed_total >= p.stop_after_stages) { ok = false; break; }
          ++armed_total;
          if (!wait_or_abort(&s->empty[stage], phase ^ 1, s, p)) { ok = false; break; }
          uint8_t* a_dst = smem + static_cast<size_t>(stage) * kStageBytes;
          mbar_arrive_expect_tx(&s->full[stage], kStageBytes);
          tma_load_2d(a_dst, &tm_x, &s->full[stage], ks * RK, T * RM);
          tma_load_2d(a_dst + kABytes, &tm_w, &s->full[stage], ks * RK, 0);
          armed |= 1u << stage;
          armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {  // let copies in flight land before the CTA's shared memory is released
        for (int i = 0; i < kStages; ++i)
          if (armed & (1u << i)) mbar_wait_bounded(&s->full[i], (armed_parity >> i) & 1u, 20000000ull);
      }
    }
  } else if (warp == kMmaWarp) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16_f32_major(RM, RN, false, false);
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int T = blockIdx.x; ok && T < total_tiles; T += grid) {
        if (!wait_or_abort(&s->tmem_empty[acc], acc_phase ^ 1, s, p)) { ok = false; break; }
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * RN);
        for (int ks = 0; ks < KS; ++ks) {
          if (!wait_or_abort(&s->full[stage], phase, s, p)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(smem + static_cast<size_t>(stage) * kStageBytes);
          const uint64_t a_desc = umma_desc_k_sw128(a_addr);
          const uint64_t b_desc = umma_desc_k_sw128(a_addr + kABytes);
#pragma unroll
          for (int k4 = 0; k4 < RK / 16; ++k4)  // 16 elements further on: 32 bytes = 2 in the 16-byte address field
            umma_bf16(d_tmem, a_desc + 2 * k4, b_desc + 2 * k4, idesc, (ks > 0 || k4 > 0) ? 1u : 0u);
          umma_commit(&s->empty[stage]);
          if (ks == KS - 1) umma_commit(&s->tmem_full[acc]);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1; }
      }
      // nothing of this CTA's tensor work may be in flight when its TMEM and shared memory go away
      if (!ok) {
        umma_commit(&s->teardown);
        mbar_wait_bounded(&s->teardown, 0, 20000000ull);
      }
    }
  } else {
    const int r = warp * 32 + lane;
    const uint32_t lane_addr = static_cast<uint32_t>(warp * 32) << 16;
    double* scr = scratch + r;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int T = blockIdx.x; T < total_tiles; T += grid) {
      if (!warp_wait_or_abort(&s->tmem_full[acc], acc_phase, s, p)) break;
      tc_fence_after_sync();
      uint32_t v[RN / 16][16];
      const uint32_t t0 = tmem_base + lane_addr + static_cast<uint32_t>(acc * RN);
#pragma unroll
      for (int c = 0; c < RN / 16; ++c) tmem_ld_x16(t0 + 16 * c, v[c]);
      tmem_ld_wait();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&s->tmem_empty[acc]);  // the row is in registers: the MMA may reuse the accumulator
      if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1; }

      // The logits leave through shared memory: the thread writes its row into the warp's boxes (16-byte
      // chunk j of a row at j ^ (row % 8), the 128-byte swizzle, so the 32 rows of a warp spread over all
      // banks) and one lane hands the boxes to TMA, which writes whole lines while the selection runs and
      // drops the rows past M and the columns past E.
      uint8_t* my_boxes = logit_tile + static_cast<size_t>(warp) * (RN / 32) * kLogitBoxBytes;
      if (lane == 0) bulk_wait_group_read_all();  // the previous tile's boxes have been read
      __syncwarp();
#pragma unroll
      for (int c = 0; c < RN / 16; ++c)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int chunk = (c & 1) * 4 + j;  // 16-byte chunk within the 128-byte row of box c / 2
          *reinterpret_cast<uint4*>(my_boxes + (c >> 1) * kLogitBoxBytes + lane * 128 + ((chunk ^ (lane & 7)) << 4)) =
              make_uint4(v[c][4 * j], v[c][4 * j + 1], v[c][4 * j + 2], v[c][4 * j + 3]);
        }
      fence_proxy_async_smem();
      __syncwarp();
      const int row0 = T * RM + warp * 32;
      if (lane == 0 && row0 < p.M) {
        for (int b = 0; b < RN / 32; ++b)
          if (32 * b < p.E) tma_store_2d(&tm_l, my_boxes + b * kLogitBoxBytes, 32 * b, row0);
        bulk_commit_group();
      }
      const int64_t row = static_cast<int64_t>(T) * RM + r;
      if (row >= p.M) continue;

      // Selection in two levels.  The row's 128 experts form eight groups of 16; each group's best not yet
      // selected expert is kept in registers.  A round picks the best of the eight candidates and then only
      // re-scans the group the winner came from -- its 16 logits are read back from the row's staged copy in
      // shared memory, because which group that is differs from lane to lane and registers cannot be indexed
      // by a run-time value.  About 150 instructions per round instead of the 770 of a scan over all experts.
      // The rule is the ascending scan's, to the letter: the first not yet selected expert stands unless a
      // later one is strictly greater (NaN or not), so ties keep the lower id.  That first expert is always in
      // group 0 (k <= 16 leaves one of its 16 unselected; with E < 16, k <= E does), so only group 0 lets its
      // first candidate stand; every other group offers only a value greater than -inf, since a NaN or -inf met
      // later in the scan could never replace the standing candidate.
      constexpr int kGroups = RN / 16;
      uint32_t taken[RN / 32];  // bit e: expert e is selected already or does not exist
#pragma unroll
      for (int w = 0; w < RN / 32; ++w) {
        const int first = p.E - 32 * w;  // experts of this word below E
        taken[w] = first >= 32 ? 0u : (first <= 0 ? 0xFFFFFFFFu : (0xFFFFFFFFu << first));
      }
      float gm[kGroups];
      int gi[kGroups];
#pragma unroll
      for (int g = 0; g < kGroups; ++g) {
        gm[g] = -INFINITY;
        gi[g] = -1;
      }
#pragma unroll
      for (int j = 0; j < 16; ++j)
#pragma unroll
        for (int g = 0; g < kGroups; ++g) {  // eight independent chains
          const int e = 16 * g + j;
          const bool avail = ((taken[e >> 5] >> (e & 31)) & 1u) == 0u;
          const float x = __uint_as_float(v[g][j]);
          const bool better = avail && ((g == 0 && gi[g] < 0) || x > gm[g]);
          gm[g] = better ? x : gm[g];
          gi[g] = better ? e : gi[g];
        }
      double mx = 0.0, den = 0.0;
      int32_t* id_out = p.ids + row * p.k;
      float* w_out = p.wts + row * p.k;
      const uint8_t* my_row = my_boxes + lane * 128;
#pragma unroll 1
      for (int rd = 0; rd < p.k; ++rd) {
        float bestv = gm[0];
        int best = gi[0];
#pragma unroll
        for (int g = 1; g < kGroups; ++g) {
          const bool better = gi[g] >= 0 && (best < 0 || gm[g] > bestv);
          bestv = better ? gm[g] : bestv;
          best = better ? gi[g] : best;
        }
        best = max(best, 0);  // k <= E leaves an expert to select in every round; never index with -1
#pragma unroll
        for (int w = 0; w < RN / 32; ++w) taken[w] |= (best >> 5) == w ? (1u << (best & 31)) : 0u;
        id_out[rd] = best;
        if (rd == 0) mx = static_cast<double>(bestv);
        const double ex = exp(static_cast<double>(bestv) - mx);
        den += ex;
        scr[rd * RM] = ex;
        if (rd + 1 < p.k) {
          // the winner's group again, from the staged row: box wg / 2, chunks 4 (wg % 2) .. + 3 at their swizzled places
          const int wg = best >> 4;
          uint32_t tw = taken[0];
#pragma unroll
          for (int w = 1; w < RN / 32; ++w) tw = (wg >> 1) == w ? taken[w] : tw;
          const uint32_t tk = tw >> ((wg & 1) * 16);
          const uint8_t* src = my_row + (wg >> 1) * kLogitBoxBytes;
          float x[16];
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            const uint4 u = *reinterpret_cast<const uint4*>(src + ((((wg & 1) * 4 + c4) ^ (lane & 7)) << 4));
            x[4 * c4] = __uint_as_float(u.x);
            x[4 * c4 + 1] = __uint_as_float(u.y);
            x[4 * c4 + 2] = __uint_as_float(u.z);
            x[4 * c4 + 3] = __uint_as_float(u.w);
          }
          // two chains of eight, then the second half's winner against the first's
          float nv[2] = {-INFINITY, -INFINITY};
          int ni[2] = {-1, -1};
#pragma unroll
          for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int jj = 8 * h + j;
              const bool avail = ((tk >> jj) & 1u) == 0u;
              const bool better = avail && ((wg == 0 && h == 0 && ni[h] < 0) || x[jj] > nv[h]);
              nv[h] = better ? x[jj] : nv[h];
              ni[h] = better ? jj : ni[h];
            }
          {
            const bool better = ni[1] >= 0 && (ni[0] < 0 || nv[1] > nv[0]);
            nv[0] = better ? nv[1] : nv[0];
            ni[0] = better ? ni[1] : ni[0];
          }
          const int ne = ni[0] >= 0 ? 16 * wg + ni[0] : -1;
#pragma unroll
          for (int g = 0; g < kGroups; ++g) {
            gm[g] = g == wg ? nv[0] : gm[g];
            gi[g] = g == wg ? ne : gi[g];
          }
        }
      }
#pragma unroll 1
      for (int rd = 0; rd < p.k; ++rd) w_out[rd] = static_cast<float>(scr[rd * RM] / den);
    }
  }

  if (warp < kEpiWarps && lane == 0) bulk_wait_group_all();  // the logits stores of this CTA are complete
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Tensor map of a row-major bf16 matrix [rows, cols]: box of 64 columns x 128 rows, 128-byte swizzle.
CUresult make_tmap(EncodeTiledFn encode, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {RK, RM};
  const cuuint32_t estr[2] = {1, 1};
  return encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

}  // namespace

bool router_fused_applies(int64_t E, int64_t k) { return E <= RN && k <= kMaxTopK; }

cudaError_t launch_router_fused(const Launch& L, EncodeTiledFn encode, const uint16_t* x, int64_t M, int64_t H,
                                const uint16_t* wr, int64_t E, int64_t k, float* logits, int32_t* ids, float* wts,
                                CUresult* cu_err) {
  *cu_err = CUDA_SUCCESS;
  if (M == 0) return cudaSuccess;
  CUtensorMap tx, tw, tl;
  CUresult r = make_tmap(encode, &tx, x, static_cast<uint64_t>(M), static_cast<uint64_t>(H));
  if (r == CUDA_SUCCESS) r = make_tmap(encode, &tw, wr, static_cast<uint64_t>(E), static_cast<uint64_t>(H));
  if (r == CUDA_SUCCESS) {  // logits fp32 [M, E]: boxes of 32 columns (128 bytes) x 32 rows
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(E), static_cast<cuuint64_t>(M)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(E) * 4};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    r = encode(&tl, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, logits, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (r != CUDA_SUCCESS) {
    *cu_err = r;
    return cudaErrorUnknown;
  }
  RouterParams p{};
  p.M = static_cast<int>(M);
  p.H = static_cast<int>(H);
  p.E = static_cast<int>(E);
  p.k = static_cast<int>(k);
  p.logits = logits;
  p.ids = ids;
  p.wts = wts;
  p.status = L.d_status;
  p.wait_limit_ns = L.wait_limit_ns ? L.wait_limit_ns : 2000000000ull;
  p.stop_after_stages = L.stop_after_stages;
  // sticky per device; atomic: contexts on several host threads may launch at once (both would set the same value)
  static std::atomic<bool> attr_set_dev[64];
  std::atomic<bool>& attr_set = attr_set_dev[L.device & 63];
  if (!attr_set.load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(router_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kSmemBytes));
    if (e != cudaSuccess) return e;
    attr_set.store(true, std::memory_order_release);
  }
  // full rounds only: with W = ceil(tiles / SMs) rounds, ceil(tiles / W) CTAs finish in W rounds
  const int64_t tiles = (M + RM - 1) / RM;
  const int64_t rounds = std::max<int64_t>(1, (tiles + L.sm_count - 1) / L.sm_count);
  const int grid = static_cast<int>(std::max<int64_t>(1, (tiles + rounds - 1) / rounds));
  ++*L.launches;
  return launch_pdl(router_fused_kernel, static_cast<unsigned>(grid), kThreads, kSmemBytes, L.stream, tx, tw, tl, p);
}

}  // namespace qarl
