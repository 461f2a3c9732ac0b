// Persistent block-scaled FP8 GEMM for sm_100a (dense projection, MoE gate_up, MoE down).
//
// Computes, for every output row m (an activation row) and column n (a weight row),
//   acc[m,n] = sum over kb ascending, from 0.0f, of  fmaf( fl(s_x[m,kb] * s_w[n/128,kb]), p_kb[m,n], acc )
// where p_kb is the tensor-core dot product of the 128 e4m3 codes of K-block kb (Sec. 2.2:
// Y ~= (s_x s_w)(X_q W_q), applied per block with fp32 accumulation).  The order is the same
// for every M, group size and tile schedule (App. C): one MMA shape (128 x 256 x 32,
// cta_group::1), four MMAs per K-block in ascending k, no split-K, no atomics.  A row's
// result depends only on that row's codes and scales and on the weight tile.
//
// A tile is 128 rows x (128 + 128) columns: two half tiles, rows [n_lo, n_lo+128) and
// [n_hi, n_hi+128) of the weight -- adjacent for linear/down, gate rows and the matching up
// rows for gate_up so that SwiGLU and the 1x128 re-quantization of h need no second pass.
//
// Structure of a CTA (512 threads = 4 warpgroups, one CTA per SM, persistent, static tile list):
//   warp 12     TMA producer: per K-block one stage = A box 128x128 B + two B boxes 128x128 B
//               (SWIZZLE_128B) into a 3-deep shared-memory ring;
//   warp 13     MMA issuer: 4 x tcgen05.mma kind::f8f6f4 per K-block into one of two
//               256-column TMEM accumulators (overwrite on the first), then tcgen05.commit to
//               free the smem stage and to publish the accumulator;
//   warps 0-7   promotion (208 registers each via setmaxnreg): warp w reads TMEM lanes
//               32*(w%4).. (its hardware quadrant) and the 64-column slice (w/4) of each half,
//               in 16-column double-buffered chunks, releases the accumulator, and adds
//               scale * partial into fp32 registers; MMA of block kb+1 overlaps promotion of kb.  At the
//               end of a tile it rounds its 128 values to bf16 into a shared-memory staging
//               tile and goes straight on to the next tile;
//   warps 8-11  epilogue: read the staged bf16 tile (coalesced, several rows per pass) and
//               finish it while the next tile's main loop runs: plain store (linear),
//               scatter by pair id (down), or SwiGLU + 1x128 amax/scale/e4m3 codes (gate_up).
//
// Every wait on an mbarrier is bounded; on expiry the thread records
// QARL_ERR_DEVICE_TIMEOUT, raises a CTA-wide abort flag that all other waits poll, and the
// CTA drains and frees its TMEM, so a broken pipeline returns an error instead of hanging.
#include <algorithm>
#include <atomic>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace qarl {
namespace {

using namespace ptx;

constexpr int BM = 128;           // rows per tile (UMMA M)
constexpr int BNH = 128;          // columns per half tile
constexpr int BN = 2 * BNH;       // UMMA N
constexpr int BK = 128;           // one K-block = one 128-byte swizzle span of e4m3
constexpr int kStages = 3;        // shared-memory ring of 48 KB stages
constexpr int kAccBufs = 2;       // TMEM accumulators of 256 columns
constexpr int kPromoWarps = 8;    // warps 0-7
constexpr int kEpiWarps = 4;      // warps 8-11
constexpr int kTmaWarp = 12;
constexpr int kMmaWarp = 13;      // and 14: two issuers; warp 15 idle (setmaxnreg works on whole warpgroups)
constexpr int kThreads = 16 * 32;
// register re-allocation: 256 x 208 + 128 x 56 + 128 x 40 = 65536 = 512 x 128 (the launch allocation)
constexpr int kPromoRegs = 208;
constexpr int kEpiRegs = 56;
constexpr int kAuxRegs = 40;
constexpr int kSliceCols = 64;    // columns of each half owned by one promotion warp
constexpr uint32_t kABytes = BM * BK;
constexpr uint32_t kBBytes = BN * BK;
constexpr uint32_t kStageBytes = kABytes + kBBytes;  // 48 KB
constexpr uint32_t kTmemCols = 512;
constexpr int kOutPitch = BN * 2 + 16;  // bytes per row of the bf16 staging tile (padded: conflict-free)
constexpr uint32_t kOutBytes = BM * kOutPitch;
constexpr int kMaxExperts = 1024;

struct GemmParams {
  const float* a_scales;
  const float* b_scales;
  const int32_t* offsets;  // [E+1] or nullptr (dense: one group of rows_total rows)
  int rows_total;
  int kblocks;             // K / 128
  int N;                   // weight rows per expert
  int E;
  int n_tiles;             // column tiles per expert
  int I;                   // gate_up: intermediate size (N = 2I)
  int early_prefetch;      // decode-sized calls: weight tiles to pull into L2 before the predecessor finishes
  uint16_t* out_bf16;
  float* out_f32;
  uint8_t* h_codes;
  float* h_scales;
  uint16_t* h_bf16;
  const int32_t* sorted_pair;
  const float* pair_weights;  // down: combine weight of each sorted position
  int* status;
  unsigned long long wait_limit_ns;
  int stop_after_stages;   // test harness only (< 0: off): the TMA producer stops arming stages after this many
};

struct __align__(8) SmemTail {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t tmem_full[kAccBufs];
  uint64_t tmem_empty[kAccBufs];
  uint64_t out_full;
  uint64_t out_empty;
  uint64_t teardown[2];
  uint32_t tmem_addr;
  int abort_flag;
  int32_t off[kMaxExperts + 1];
  int32_t prefix[kMaxExperts + 1];
};

constexpr size_t kSmemBytes = 1024 + static_cast<size_t>(kStages) * kStageBytes + kOutBytes + sizeof(SmemTail);
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

struct TileCoord {
  int e, n_tile, m0, m_end;
};

// Tile T -> (expert, column tile, first row, end of the expert's rows).  Within an expert the
// row tiles vary fastest, so CTAs running at the same time share one weight tile through L2.
__device__ __forceinline__ TileCoord decode_tile(const SmemTail* s, int T, int& cur_e) {
  while (T >= s->prefix[cur_e + 1]) ++cur_e;
  const int local = T - s->prefix[cur_e];
  const int rows = s->off[cur_e + 1] - s->off[cur_e];
  const int m_tiles = (rows + BM - 1) / BM;
  TileCoord c;
  c.e = cur_e;
  c.n_tile = local / m_tiles;
  c.m0 = s->off[cur_e] + (local % m_tiles) * BM;
  c.m_end = s->off[cur_e + 1];
  return c;
}

// Bounded wait of one thread.  False: the limit ran out here (the error is recorded and the
// CTA-wide abort flag raised) or another thread raised the flag; the caller leaves its loop.
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, SmemTail* s, const GemmParams& p) {
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

// The same for a whole warp: every lane polls (one polling lane with 31 parked at a shuffle
// measured 2x slower on the short-K down projection), then the lanes vote, so all 32 take the
// same branch and the warp-wide shuffles and barriers that follow never see a split warp
// (lanes polling on their own could disagree when a barrier completes right at the limit).
__device__ __forceinline__ bool warp_wait_or_abort(uint64_t* bar, uint32_t parity, SmemTail* s, const GemmParams& p) {
  return __all_sync(0xFFFFFFFFu, wait_or_abort(bar, parity, s, p) ? 1 : 0) != 0;
}

// silu(g) * u in fp32 with the fast exp and reciprocal (relative error ~1e-6, far below the
// half-ulp of the bf16 the result is rounded to).
__device__ __forceinline__ float silu_mul(float g, float u) {
  return __fdividef(g, 1.0f + __expf(-g)) * u;
}

// acc[j] = fmaf(sc, v[j], acc[j]) for 16 values (8 float2 accumulators).
__device__ __forceinline__ void promote16(float2* acc, const uint32_t (&v)[16], float sc) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    acc[j].x = __fmaf_rn(sc, __uint_as_float(v[2 * j]), acc[j].x);
    acc[j].y = __fmaf_rn(sc, __uint_as_float(v[2 * j + 1]), acc[j].y);
  }
}

__device__ __forceinline__ uint32_t bf16x2_bits(float lo, float hi) {
  const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);  // .x = lo (low 16 bits), .y = hi
  return *reinterpret_cast<const uint32_t*>(&b);
}

template <int MODE>
__global__ void __launch_bounds__(kThreads, 1)
gemm_blockscaled_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                        const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* out_tile = smem + static_cast<size_t>(kStages) * kStageBytes;
  SmemTail* s = reinterpret_cast<SmemTail*>(out_tile + kOutBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- set-up: barriers, TMEM, tile list ------------------------------------------------
  pdl_trigger();
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&s->full[i], 1);
      mbar_init(&s->empty[i], 1);
    }
    for (int i = 0; i < kAccBufs; ++i) {
      mbar_init(&s->tmem_full[i], 1);
      mbar_init(&s->tmem_empty[i], kPromoWarps);
    }
    mbar_init(&s->out_full, kPromoWarps);
    mbar_init(&s->out_empty, kEpiWarps);
    mbar_init(&s->teardown[0], 1);
    mbar_init(&s->teardown[1], 1);
    s->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kTmaWarp && lane == 0) {
    prefetch_tensormap(&tm_a);
    prefetch_tensormap(&tm_b);
  }
  if (warp == kMmaWarp) {
    tmem_alloc(&s->tmem_addr, kTmemCols);
    tmem_relinquish();
  }
  if (warp == kTmaWarp && lane == 0 && p.early_prefetch > 0) {
    // Decode-sized calls are bound by streaming the weights from HBM, and the kernels before
    // this one in the stream (permute, activation quantization) leave the memory system idle.
    // The weights do not depend on them, so pull this CTA's first weight tiles into L2 now.
    // Tile T is guessed as (expert T / n_tiles, column tile T % n_tiles), exact when every
    // expert has one row tile; a wrong guess only costs an unused L2 fill.
    for (int t = 0; t < p.early_prefetch; ++t) {
      const int T = blockIdx.x + t * gridDim.x;
      if (T >= p.E * p.n_tiles) break;
      const int e = T / p.n_tiles, n_tile = T % p.n_tiles;
      int row_lo, row_hi;
      if (MODE == kModeGateUp) {
        row_lo = e * p.N + n_tile * BNH;
        row_hi = row_lo + p.I;
      } else {
        row_lo = e * p.N + n_tile * BN;
        row_hi = row_lo + BNH;
      }
      for (int kb = 0; kb < p.kblocks; ++kb) {
        tma_prefetch_2d(&tm_b, kb * BK, row_lo);
        tma_prefetch_2d(&tm_b, kb * BK, row_hi);
      }
    }
  }
  pdl_wait();  // everything above read no data of the predecessor; from here on its results are needed
  // Group boundaries, forced into [0, rows_total]: whatever the caller's array holds, no tile
  // and no store mask derived from it can reach outside the tensors.
  for (int e = threadIdx.x; e <= p.E; e += kThreads) {
    const int raw = p.offsets ? p.offsets[e] : (e == 0 ? 0 : p.rows_total);
    const int v = min(max(raw, 0), p.rows_total);
    if (v != raw) set_status(p.status, QARL_ERR_INVALID_ARG);
    s->off[e] = v;
  }
  __syncthreads();
  if (warp == 0) {
    // exclusive scan of tiles per expert
    int carry = 0;
    for (int base = 0; base < p.E; base += 32) {
      const int e = base + lane;
      int v = 0;
      if (e < p.E) {
        // a group that ends before it starts (offsets out of order) is reported and gets no tile;
        // with every boundary inside [0, rows_total] the other groups stay inside the tensors
        const int rows = s->off[e + 1] - s->off[e];
        if (rows < 0) set_status(p.status, QARL_ERR_INVALID_ARG);
        v = ((max(rows, 0) + BM - 1) / BM) * p.n_tiles;
      }
      int inc = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += u;
      }
      if (e < p.E) s->prefix[e] = carry + inc - v;
      carry += __shfl_sync(0xFFFFFFFFu, inc, 31);
    }
    if (lane == 0) s->prefix[p.E] = carry;
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = s->tmem_addr;
  const int total_tiles = s->prefix[p.E];
  // Balance the static schedule: with W = ceil(tiles / CTAs) rounds, ceil(tiles / W) CTAs already
  // finish in W rounds; using exactly that many keeps every round full (768 decode tiles: 128 CTAs
  // x 6 instead of 148 CTAs of which 120 idle through the sixth round) and leaves the streaming
  // bandwidth to the CTAs that still have work.  The CTAs beyond that count retire at once.
  int num_ctas = gridDim.x;
  if (total_tiles > 0) {
    const int rounds = (total_tiles + num_ctas - 1) / num_ctas;
    num_ctas = (total_tiles + rounds - 1) / rounds;
  }
  const int first_tile = static_cast<int>(blockIdx.x) < num_ctas ? static_cast<int>(blockIdx.x) : total_tiles;
  const int KB = p.kblocks;
  const int NB = p.N / BNH;  // weight scale block-rows per expert

  if (warp >= kPromoWarps + kEpiWarps) setmaxnreg_dec<kAuxRegs>();
  else if (warp >= kPromoWarps) setmaxnreg_dec<kEpiRegs>();
  else setmaxnreg_inc<kPromoRegs>();
  if (warp >= kPromoWarps + kEpiWarps) {
    if (warp == kTmaWarp) {
      // =============================== TMA producer =====================================
      if (lane == 0) {
        int stage = 0;
        uint32_t phase = 0;
        uint32_t armed = 0, armed_parity = 0;  // per-stage: has a load in flight / its parity
        int armed_total = 0;
        int cur_e = 0;
        bool ok = true;
        // weight rows of a tile's two halves
        auto b_rows = [&](const TileCoord& c, int& row_lo, int& row_hi) {
          if (MODE == kModeGateUp) {
            row_lo = c.e * p.N + c.n_tile * BNH;
            row_hi = row_lo + p.I;
          } else {
            row_lo = c.e * p.N + c.n_tile * BN;
            row_hi = row_lo + BNH;
          }
        };
        for (int T = first_tile; ok && T < total_tiles; T += num_ctas) {
          const TileCoord c = decode_tile(s, T, cur_e);
          int row_lo, row_hi;
          b_rows(c, row_lo, row_hi);
          for (int kb = 0; kb < KB; ++kb) {
            if (p.stop_after_stages >= 0 && armed_total >= p.stop_after_stages) { ok = false; break; }
            ++armed_total;
            if (!wait_or_abort(&s->empty[stage], phase ^ 1, s, p)) { ok = false; break; }
            uint8_t* a_dst = smem + static_cast<size_t>(stage) * kStageBytes;
            uint8_t* b_dst = a_dst + kABytes;
            mbar_arrive_expect_tx(&s->full[stage], kStageBytes);
            tma_load_2d(a_dst, &tm_a, &s->full[stage], kb * BK, c.m0);
            tma_load_2d(b_dst, &tm_b, &s->full[stage], kb * BK, row_lo);
            tma_load_2d(b_dst + kBBytes / 2, &tm_b, &s->full[stage], kb * BK, row_hi);
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
    } else if (warp == kMmaWarp || warp == kMmaWarp + 1) {
      // =============================== MMA issuers ======================================
      // Two threads, one per TMEM accumulator: K-block n of this CTA (counted across its tiles) is
      // issued by thread n % 2 into accumulator n % 2.  Every K-block starts a fresh accumulator, so
      // the two never write the same columns, and the fixed cost per K-block of one thread waiting,
      // issuing and committing (about as long as the MMAs themselves take) is spread over two.
      if (lane == 0) {
        constexpr uint32_t idesc = umma_idesc_e4m3_f32(BM, BN);
        const int me = warp - kMmaWarp;
        uint32_t n = 0;  // K-blocks of this CTA so far
        bool ok = true;
        for (int T = first_tile; ok && T < total_tiles; T += num_ctas) {
          for (int kb = 0; kb < KB; ++kb, ++n) {
            if (static_cast<int>(n & 1u) != me) continue;
            const uint32_t stage = n % kStages, phase = (n / kStages) & 1u;
            const uint32_t ks = n & 1u, acc_phase = (n >> 1) & 1u;
            if (!wait_or_abort(&s->tmem_empty[ks], acc_phase ^ 1, s, p)) { ok = false; break; }
            if (!wait_or_abort(&s->full[stage], phase, s, p)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t a_addr = smem_u32(smem + static_cast<size_t>(stage) * kStageBytes);
            const uint64_t a_desc = umma_desc_k_sw128(a_addr);
            const uint64_t b_desc = umma_desc_k_sw128(a_addr + kABytes);
            const uint32_t d_tmem = tmem_base + ks * BN;
#pragma unroll
            for (int k4 = 0; k4 < BK / 32; ++k4)  // +32 bytes of K = +2 in the 16-byte address field
              umma_f8(d_tmem, a_desc + 2 * k4, b_desc + 2 * k4, idesc, k4 > 0 ? 1u : 0u);
            umma_commit(&s->empty[stage]);
            umma_commit(&s->tmem_full[ks]);
          }
        }
        // Nothing of this CTA's tensor work may be in flight when its TMEM and shared memory
        // go away: after a normal run every MMA has been consumed already; after an abort
        // some may still be executing, so wait (bounded) for all of them.
        if (!ok) {
          umma_commit(&s->teardown[me]);
          mbar_wait_bounded(&s->teardown[me], 0, 20000000ull);
        }
      }
    }
  } else if (warp >= kPromoWarps) {
    // =============================== epilogue warps ===================================
    const int ew = warp - kPromoWarps;
    int cur_e = 0;
    uint32_t tile_iter = 0;
    for (int T = first_tile; T < total_tiles; T += num_ctas, ++tile_iter) {
      const TileCoord c = decode_tile(s, T, cur_e);
      int my_pair = 0;  // down: destination (flat pair id) of the lane-th row this warp handles
      if (MODE == kModeDown) {
        const int row = c.m0 + ew + kEpiWarps * lane;
        // no pair map: the contribution stays at its sorted position (expert-parallel use)
        if (row < c.m_end)
          my_pair = p.sorted_pair ? min(max(__ldg(p.sorted_pair + row), 0), p.rows_total - 1) : row;  // in bounds even after bad ids
      }
      if (!warp_wait_or_abort(&s->out_full, tile_iter & 1u, s, p)) break;
      if (MODE == kModeGateUp) {
        // 8 lanes per row, 4 rows per pass.  Lane `sub` owns h columns [8 sub, 8 sub + 8) and
        // [64 + 8 sub, 64 + 8 sub + 8) of the row's 128-wide quantization group, so that a
        // quarter-warp reads 128 contiguous bytes of the staging tile (conflict-free).
        const int sub = lane & 7, rsel = lane >> 3;
        const int IB = p.I / BNH;
#pragma unroll 2
        for (int i = 0; i < BM / (kEpiWarps * 4); ++i) {
          const int r0 = (i * kEpiWarps + ew) * 4;
          if (c.m0 + r0 >= c.m_end) break;  // warp-uniform: rows ascend with i
          const int rr = r0 + rsel;
          const int row = c.m0 + rr;
          const bool live = row < c.m_end;
          const uint8_t* src = out_tile + rr * kOutPitch + sub * 16;
          uint4 g[2], u[2];
          g[0] = *reinterpret_cast<const uint4*>(src);
          g[1] = *reinterpret_cast<const uint4*>(src + 128);
          u[0] = *reinterpret_cast<const uint4*>(src + BNH * 2);
          u[1] = *reinterpret_cast<const uint4*>(src + BNH * 2 + 128);
          uint32_t hb[8];
          uint32_t m = 0;
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            const uint32_t gw[4] = {g[t].x, g[t].y, g[t].z, g[t].w};
            const uint32_t uw[4] = {u[t].x, u[t].y, u[t].z, u[t].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float h0 = silu_mul(bf16_bits_to_f32(gw[j] & 0xFFFFu), bf16_bits_to_f32(uw[j] & 0xFFFFu));
              const float h1 = silu_mul(__uint_as_float(gw[j] & 0xFFFF0000u), __uint_as_float(uw[j] & 0xFFFF0000u));
              hb[4 * t + j] = bf16x2_bits(h0, h1);
              m = __vmaxu2(m, hb[4 * t + j] & 0x7FFF7FFFu);  // |bf16| bit patterns: exact, order-free max
            }
          }
          m = max(m & 0xFFFFu, m >> 16);
#pragma unroll
          for (int o = 4; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
          float inv;
          const float sc = block_scale(bf16_bits_to_f32(m), &inv);
          uint32_t cw[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t x0 = hb[2 * j], x1 = hb[2 * j + 1];
            cw[j] = cvt_e4m3x4(__fmul_rn(bf16_bits_to_f32(x0 & 0xFFFFu), inv), __fmul_rn(__uint_as_float(x0 & 0xFFFF0000u), inv),
                               __fmul_rn(bf16_bits_to_f32(x1 & 0xFFFFu), inv), __fmul_rn(__uint_as_float(x1 & 0xFFFF0000u), inv));
          }
          if (live) {
            const int col = c.n_tile * BNH + 8 * sub;
            uint8_t* hc = p.h_codes + static_cast<int64_t>(row) * p.I + col;
            *reinterpret_cast<uint2*>(hc) = make_uint2(cw[0], cw[1]);
            *reinterpret_cast<uint2*>(hc + 64) = make_uint2(cw[2], cw[3]);
            if (sub == 0) p.h_scales[static_cast<int64_t>(row) * IB + c.n_tile] = sc;
            if (p.h_bf16) {
              uint16_t* hd = p.h_bf16 + static_cast<int64_t>(row) * p.I + col;
              *reinterpret_cast<uint4*>(hd) = make_uint4(hb[0], hb[1], hb[2], hb[3]);
              *reinterpret_cast<uint4*>(hd + 64) = make_uint4(hb[4], hb[5], hb[6], hb[7]);
            }
            if (p.out_bf16) {  // debug dump of the bf16 gate_up row
              uint16_t* gd = p.out_bf16 + static_cast<int64_t>(row) * p.N + col;
              *reinterpret_cast<uint4*>(gd) = g[0];
              *reinterpret_cast<uint4*>(gd + 64) = g[1];
              *reinterpret_cast<uint4*>(gd + p.I) = u[0];
              *reinterpret_cast<uint4*>(gd + p.I + 64) = u[1];
            }
          }
        }
      } else {
        // the tile's 256 columns are contiguous in the output row: 512 bytes per row, 16 per lane
        const int col = c.n_tile * BN + 8 * lane;
        const bool col_ok = col < p.N;
#pragma unroll 4
        for (int i = 0; i < BM / kEpiWarps; ++i) {
          const int rr = ew + kEpiWarps * i;
          const int row = c.m0 + rr;
          if (row >= c.m_end) break;
          const uint4 v = *reinterpret_cast<const uint4*>(out_tile + rr * kOutPitch + lane * 16);
          int64_t out_row = row;
          if (MODE == kModeDown) out_row = __shfl_sync(0xFFFFFFFFu, my_pair, i);  // lane i holds row i's pair id
          if (col_ok) *reinterpret_cast<uint4*>(p.out_bf16 + out_row * p.N + col) = v;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&s->out_empty);
    }
  } else {
    // =============================== promotion warps ==================================
    const int q = warp & 3;          // TMEM lane quadrant this warp may read
    const int hs = warp >> 2;        // which 64-column slice of each half tile
    const int r = q * 32 + lane;     // row within the tile
    const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
    int ks = 0;
    uint32_t acc_phase = 0;
    int cur_e = 0;
    uint32_t tile_iter = 0;

    // scale pointers of a tile for this thread's row: s_x[row, :], s_w[lo block-row, :] and
    // the offset from the lo to the hi block-row
    auto scale_ptrs = [&](const TileCoord& c, const float*& sx, const float*& swl, int& hi_off) {
      const int row_c = min(c.m0 + r, p.rows_total - 1);
      int nb_lo, nb_hi;
      if (MODE == kModeGateUp) {
        nb_lo = c.n_tile;
        nb_hi = c.n_tile + p.I / BNH;
      } else {
        nb_lo = 2 * c.n_tile;
        nb_hi = min(2 * c.n_tile + 1, NB - 1);
      }
      sx = p.a_scales + static_cast<int64_t>(row_c) * KB;
      swl = p.b_scales + (static_cast<int64_t>(c.e) * NB + nb_lo) * KB;
      hi_off = (nb_hi - nb_lo) * KB;
    };

    int T = first_tile;
    if (T < total_tiles) {
      TileCoord c = decode_tile(s, T, cur_e);
      const float *sx_ptr, *sw_lo_ptr;
      int sw_hi_off;
      scale_ptrs(c, sx_ptr, sw_lo_ptr, sw_hi_off);
      float sx_next = __ldg(sx_ptr), swl_next = __ldg(sw_lo_ptr), swh_next = __ldg(sw_lo_ptr + sw_hi_off);
      bool ok = true;
      for (;;) {
        const int row = c.m0 + r;
        const bool valid = row < c.m_end;
        // a warp whose 32 rows all lie past the group's end (ragged tails, decode-sized groups)
        // keeps the barrier protocol going but reads and accumulates nothing
        const bool warp_live = c.m0 + q * 32 < c.m_end;
        const int Tn = T + num_ctas;
        const bool has_next = Tn < total_tiles;
        TileCoord cn = c;
        float w = 0.0f;  // down: the pair's combine weight (sorted order), used at the end of the tile
        if (MODE == kModeDown && valid) w = __ldg(p.pair_weights + row);

        float2 acc_lo[32], acc_hi[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) acc_lo[j] = acc_hi[j] = make_float2(0.0f, 0.0f);

        for (int kb = 0; kb < KB; ++kb) {
          const float sc_lo = __fmul_rn(sx_next, swl_next);
          const float sc_hi = __fmul_rn(sx_next, swh_next);
          if (kb + 1 < KB) {
            sx_next = __ldg(sx_ptr + kb + 1);
            swl_next = __ldg(sw_lo_ptr + kb + 1);
            swh_next = __ldg(sw_lo_ptr + sw_hi_off + kb + 1);
          } else if (has_next) {  // first scales of the next tile: their latency hides behind this block
            cn = decode_tile(s, Tn, cur_e);
            scale_ptrs(cn, sx_ptr, sw_lo_ptr, sw_hi_off);
            sx_next = __ldg(sx_ptr);
            swl_next = __ldg(sw_lo_ptr);
            swh_next = __ldg(sw_lo_ptr + sw_hi_off);
          }
          if (!warp_wait_or_abort(&s->tmem_full[ks], acc_phase, s, p)) { ok = false; break; }
          tc_fence_after_sync();
          if (!warp_live) {
            tc_fence_before_sync();
            if (lane == 0) mbar_arrive(&s->tmem_empty[ks]);
          } else {
            const uint32_t t0 = tmem_base + lane_addr + static_cast<uint32_t>(ks * BN + hs * kSliceCols);
            // 16-column chunks, double-buffered: the load of chunk c+1 is in flight while chunk c
            // is accumulated; small enough that nothing spills under the register budget.
            uint32_t va[16], vb[16];
            tmem_ld_x16(t0, va);
            tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const uint32_t next = (c < 3) ? t0 + 16 * (c + 1) : t0 + BNH;
              if (c & 1) { tmem_ld_x16(next, va); promote16(acc_lo + 8 * c, vb, sc_lo); }
              else       { tmem_ld_x16(next, vb); promote16(acc_lo + 8 * c, va, sc_lo); }
              tmem_ld_wait();
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              if (c < 3) {
                if (c & 1) tmem_ld_x16(t0 + BNH + 16 * (c + 1), va);
                else       tmem_ld_x16(t0 + BNH + 16 * (c + 1), vb);
              }
              if (c & 1) promote16(acc_hi + 8 * c, vb, sc_hi);
              else       promote16(acc_hi + 8 * c, va, sc_hi);
              if (c < 3) tmem_ld_wait();
              if (c == 2) {
                // (the last chunk is in registers after this wait): this warp's reads of the
                // accumulator are done, hand it back to the MMA warp
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&s->tmem_empty[ks]);
              }
            }
          }
          if (++ks == kAccBufs) { ks = 0; acc_phase ^= 1; }
        }
        if (!ok) break;

        // ---- hand the tile to the epilogue warps as bf16 -----------------------------------
        if ((MODE == kModeLinear || MODE == kModeDown) && p.out_f32 && valid) {  // debug fp32 dump
          const int col_lo = c.n_tile * BN + hs * kSliceCols;
          const int col_hi = col_lo + BNH;
          float2* d_lo = reinterpret_cast<float2*>(p.out_f32 + static_cast<int64_t>(row) * p.N + col_lo);
          float2* d_hi = reinterpret_cast<float2*>(p.out_f32 + static_cast<int64_t>(row) * p.N + col_hi);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            d_lo[j] = acc_lo[j];
            if (col_hi < p.N) d_hi[j] = acc_hi[j];
          }
        }
        if (MODE == kModeDown) {  // contribution = bf16( fl(w * y) )
          const float2 w2 = make_float2(w, w);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            acc_lo[j] = __fmul2_rn(w2, acc_lo[j]);
            acc_hi[j] = __fmul2_rn(w2, acc_hi[j]);
          }
        }
        if (!warp_wait_or_abort(&s->out_empty, (tile_iter & 1u) ^ 1u, s, p)) break;  // previous tile drained
        if (warp_live) {
          uint4* d_lo = reinterpret_cast<uint4*>(out_tile + r * kOutPitch + hs * (kSliceCols * 2));
          uint4* d_hi = reinterpret_cast<uint4*>(out_tile + r * kOutPitch + BNH * 2 + hs * (kSliceCols * 2));
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            d_lo[j] = make_uint4(bf16x2_bits(acc_lo[4 * j].x, acc_lo[4 * j].y), bf16x2_bits(acc_lo[4 * j + 1].x, acc_lo[4 * j + 1].y),
                                 bf16x2_bits(acc_lo[4 * j + 2].x, acc_lo[4 * j + 2].y), bf16x2_bits(acc_lo[4 * j + 3].x, acc_lo[4 * j + 3].y));
            d_hi[j] = make_uint4(bf16x2_bits(acc_hi[4 * j].x, acc_hi[4 * j].y), bf16x2_bits(acc_hi[4 * j + 1].x, acc_hi[4 * j + 1].y),
                                 bf16x2_bits(acc_hi[4 * j + 2].x, acc_hi[4 * j + 2].y), bf16x2_bits(acc_hi[4 * j + 3].x, acc_hi[4 * j + 3].y));
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&s->out_full);
        if (!has_next) break;
        T = Tn;
        c = cn;
        ++tile_iter;
      }
    }
  }

  // ---- teardown ---------------------------------------------------------------------------
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace


namespace {

CUresult make_tmap(EncodeTiledFn encode, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols) {
  // u8 tensor [rows, cols] row-major; box = 128 bytes x 128 rows, 128-byte swizzle, zero fill.
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols};
  const cuuint32_t box[2] = {BK, BM};
  const cuuint32_t estr[2] = {1, 1};
  return encode(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

template <int MODE>
cudaError_t launch_mode(const Launch& L, const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p,
                        int grid) {
  // sticky per function and device; atomic: contexts on several host threads may launch at once (both
  // would set the same value)
  static std::atomic<bool> attr_set_dev[64];
  std::atomic<bool>& attr_set = attr_set_dev[L.device & 63];
  if (!attr_set.load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_blockscaled_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kSmemBytes));
    if (e != cudaSuccess) return e;
    attr_set.store(true, std::memory_order_release);
  }
  ++*L.launches;
  return launch_pdl(gemm_blockscaled_kernel<MODE>, static_cast<unsigned>(grid), kThreads, kSmemBytes, L.stream, ta, tb, p);
}

}  // namespace

cudaError_t launch_gemm(const Launch& L, EncodeTiledFn encode, const GemmArgs& a, CUresult* cu_err) {
  *cu_err = CUDA_SUCCESS;
  if (a.rows_total == 0) return cudaSuccess;
  // decode-sized groups: the swapped-operand kernel (bitwise the same rows, bound by the weight stream)
  if (L.gemm_path == 2 ? ((a.offsets != nullptr || a.E == 1) && a.K / BK <= 64) : (L.gemm_path == 0 && gemm_decode_applies(a)))
    return launch_gemm_decode(L, encode, a, cu_err);
  CUtensorMap ta, tb;
  CUresult r = make_tmap(encode, &ta, a.a_codes, static_cast<uint64_t>(a.rows_total), static_cast<uint64_t>(a.K));
  if (r == CUDA_SUCCESS)
    r = make_tmap(encode, &tb, a.b_codes, static_cast<uint64_t>(a.E * a.N), static_cast<uint64_t>(a.K));
  if (r != CUDA_SUCCESS) {
    *cu_err = r;
    return cudaErrorUnknown;
  }
  GemmParams p{};
  p.a_scales = a.a_scales;
  p.b_scales = a.b_scales;
  p.offsets = a.offsets;
  p.rows_total = static_cast<int>(a.rows_total);
  p.kblocks = static_cast<int>(a.K / BK);
  p.N = static_cast<int>(a.N);
  p.E = static_cast<int>(a.E);
  p.I = static_cast<int>(a.N / 2);
  p.n_tiles = a.mode == kModeGateUp ? static_cast<int>(a.N / 2 / BNH) : static_cast<int>((a.N + BN - 1) / BN);
  p.out_bf16 = a.out_bf16;
  p.out_f32 = a.out_f32;
  p.h_codes = a.h_codes;
  p.h_scales = a.h_scales;
  p.h_bf16 = a.h_bf16;
  p.sorted_pair = a.sorted_pair;
  p.pair_weights = a.pair_weights;
  p.status = L.d_status;
  p.wait_limit_ns = L.wait_limit_ns ? L.wait_limit_ns : 2000000000ull;
  p.stop_after_stages = L.stop_after_stages;
  // decode-sized call (at most one row tile per expert): see the early prefetch in the kernel
  if (a.rows_total <= a.E * BM) {
    const int64_t tile_bytes = static_cast<int64_t>(p.kblocks) * kBBytes;
    const int64_t budget = 80ll << 20;  // stay well inside the 126 MB L2
    p.early_prefetch = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(3, budget / (tile_bytes * L.sm_count))));
  }
  // upper bound on the tile count (group sizes live on the device): each expert adds at most
  // one partial row tile
  const int64_t m_tiles_max = a.rows_total / BM + a.E;
  const int grid = static_cast<int>(std::min<int64_t>(L.sm_count, m_tiles_max * p.n_tiles));
  switch (a.mode) {
    case kModeLinear: return launch_mode<kModeLinear>(L, ta, tb, p, grid);
    case kModeGateUp: return launch_mode<kModeGateUp>(L, ta, tb, p, grid);
    case kModeDown: return launch_mode<kModeDown>(L, ta, tb, p, grid);
  }
  return cudaErrorInvalidValue;
}

}  // namespace qarl
