// Persistent W4A16 GEMM for sm_100a (dense projection, MoE gate_up, MoE down): bf16 activations
// times 4-bit group-quantized weights (Sec. 2.2, integer quantization; the format of the
// paper's larger MoE models, Sec. 3.1).
//
//   y[m,n] = sum_k x[m,k] * w^[n,k],   w^ = bf16( s * (W_q - z) )   (Dequant of Sec. 2.2)
//
// with one (s, z) per 128 K-elements of a weight row, s a bf16 value.  The weights cross HBM
// and L2 as 4-bit codes only; they are expanded to bf16 in shared memory, next to the tensor
// core, and the whole K reduction of a tile accumulates in TMEM (fp32) in ascending k, one MMA
// shape, no split-K: a row's result depends on that row and the weight tile only, never on the
// batch around it (App. C).
//
// A tile is 128 rows x (128 + 128) columns, as in the FP8 kernel: the two halves are adjacent
// weight rows for linear/down, gate rows and the matching up rows for gate_up (SwiGLU in the
// epilogue).  One K-step is 64 elements = one 128-byte swizzle span of bf16.
//
// Structure of a CTA (704 threads, one CTA per SM, persistent, static tile list):
//   warp 20     TMA producer: per K-step the A box (128 rows x 64 bf16, SWIZZLE_128B) and two
//               4 KB chunks of packed codes (128 weight rows x 64 K-elements each, contiguous
//               in the tile-major weight storage: one bulk copy per half) into a ring of load stages;
//   warps 4-19  dequantization, two groups of 8 warps on alternate K-steps: thread n owns weight row n of the tile; it reads its 32 bytes
//               of codes, forms pairs (w >> 4j) & 0x000F000F | 0x43004300 = bf16x2 (128 + q),
//               subtracts 128 + z (exact), multiplies by s (one rounding: the bf16 of the exact
//               product), and writes the 128-byte row of the bf16 B tile in the 128-byte swizzle
//               the tensor core expects; a proxy fence, then the warp arrives on the stage;
//   warp 21     MMA issuer: 4 x tcgen05.mma kind::f16 (128 x 256 x 16) per K-step into one of
//               two 256-column TMEM accumulators; tcgen05.commit frees the stages, and after
//               the last K-step publishes the accumulator;
//   warps 0-3   epilogue: TMEM -> registers -> bf16 output (linear), SwiGLU -> h (gate_up),
//               weight * y -> contribution by pair id (down), while the next tile's main loop
//               runs on the other accumulator.
//
// Every wait on an mbarrier is bounded; on expiry the thread records QARL_ERR_DEVICE_TIMEOUT,
// raises a CTA-wide abort flag that all other waits poll, and the CTA drains and frees its TMEM.
#include <algorithm>
#include <atomic>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "sched.cuh"
#include "w4_dequant.cuh"

namespace qarl {
namespace {

using namespace ptx;

constexpr int BM = 128;            // rows per tile (UMMA M)
constexpr int BNH = 128;           // columns per half tile
constexpr int BN = 2 * BNH;        // UMMA N
constexpr int BK = 64;             // bf16 elements per K-step (128 bytes)
constexpr int kEpiWarps = 4;       // warps 0-3 (TMEM quadrant = warp index)
constexpr int kDqGroupWarps = 8;   // one warp per 32 weight rows of the tile
constexpr int kDqGroups = 2;       // warps 4-11 expand the even K-steps, warps 12-19 the odd ones
constexpr int kDqWarps = kDqGroups * kDqGroupWarps;
constexpr int kTmaWarp = 20;
constexpr int kMmaWarp = 21;
constexpr int kThreads = 22 * 32;
constexpr uint32_t kAHalfBytes = BM * BK * 2;    // 16 KB: 128 token rows x 64 bf16
constexpr uint32_t kQHalfBytes = BNH * BK / 2;   // 4 KB: 128 rows x 32 bytes of codes
constexpr uint32_t kQBytes = 2 * kQHalfBytes;    // 8 KB
constexpr uint32_t kDqBytes = BN * BK * 2;       // 32 KB
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxExperts = 1024;

// A tile holds MT x 128 token rows.  MT = 2 (training-sized groups) expands every weight tile
// once for 256 rows -- half the shared-memory traffic per flop, which is what bounds this
// kernel -- at the price of a single set of accumulators (the epilogue, ~2% of a tile, is not
// overlapped).  MT = 1 (decode-sized groups) keeps two accumulator sets and wastes no MMA work
// on rows that do not exist.
// Codes ring: always an even number of stages, so each dequantization group meets only stages it
// consumed itself the time before (a parity wait cannot tell two outstanding fills apart).
constexpr int kQStages = 4;
template <int MT>
struct Cfg {
  static constexpr int kRows = MT * BM;
  static constexpr uint32_t kABytes = MT * kAHalfBytes;
  static constexpr int kAStages = MT == 1 ? 4 : 3;      // token tiles (ring of its own, freed by the MMA)
  static constexpr int kDqStages = MT == 1 ? 3 : 2;     // dequantized B tiles
  static constexpr int kAccBufs = MT == 1 ? 2 : 1;      // sets of MT 256-column TMEM accumulators
  static constexpr size_t kSmemBytes = 1024 + static_cast<size_t>(kAStages) * kABytes +
                                       static_cast<size_t>(kQStages) * kQBytes +
                                       static_cast<size_t>(kDqStages) * kDqBytes;
};
constexpr int kMaxAStages = 4, kMaxDqStages = 3, kMaxAccBufs = 2;

struct W4Params {
  const uint8_t* b_packed;   // tile-major 4 KB chunks [E][N/128][K/64]
  const uint16_t* b_scales;  // bf16 bits [E][K/128][N]
  const uint8_t* b_zeros;    // [E][K/128][N]
  const int32_t* offsets;
  int rows_total;
  int ksteps;                // K / 64
  int N;
  int E;
  int n_tiles;
  int I;
  uint16_t* out_bf16;
  float* out_f32;
  uint16_t* h_bf16;
  const int32_t* sorted_pair;
  const float* pair_weights;
  int* status;
  unsigned long long wait_limit_ns;
};

struct __align__(8) SmemTail {
  uint64_t a_full[kMaxAStages];
  uint64_t a_empty[kMaxAStages];
  uint64_t q_full[kQStages];
  uint64_t q_empty[kQStages];
  uint64_t dq_full[kMaxDqStages];
  uint64_t dq_empty[kMaxDqStages];
  uint64_t tmem_full[kMaxAccBufs];
  uint64_t tmem_empty[kMaxAccBufs];
  uint64_t teardown;
  uint32_t tmem_addr;
  int abort_flag;
  int32_t off[kMaxExperts + 1];
  int32_t prefix[kMaxExperts + 1];
};

template <int MT>
constexpr size_t smem_bytes() { return Cfg<MT>::kSmemBytes + sizeof(SmemTail); }
static_assert(smem_bytes<1>() <= 227 * 1024 && smem_bytes<2>() <= 227 * 1024, "shared memory budget");

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, SmemTail* s, const W4Params& p) {
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

// The same for a whole warp: every lane polls, then the lanes vote, so all 32 take the same
// branch and the warp-wide operations that follow never see a split warp (lanes polling on
// their own could disagree when a barrier completes right at the limit).
__device__ __forceinline__ bool warp_wait_or_abort(uint64_t* bar, uint32_t parity, SmemTail* s, const W4Params& p) {
  return __all_sync(0xFFFFFFFFu, wait_or_abort(bar, parity, s, p) ? 1 : 0) != 0;
}

__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

__device__ __forceinline__ uint32_t bf16x2_bits(float lo, float hi) {
  const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&b);
}

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

template <int MODE, int MT, int FMT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_w4a16_kernel(const __grid_constant__ CUtensorMap tm_a, const W4Params p) {
  using C = Cfg<MT>;
  constexpr int kAStages = C::kAStages, kDqStages = C::kDqStages, kAccBufs = C::kAccBufs;
  constexpr uint32_t kABytes = C::kABytes;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_base = smem + static_cast<size_t>(kAStages) * kABytes;
  uint8_t* dq_base = q_base + static_cast<size_t>(kQStages) * kQBytes;
  SmemTail* s = reinterpret_cast<SmemTail*>(dq_base + static_cast<size_t>(kDqStages) * kDqBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- set-up: barriers, TMEM, tile list ------------------------------------------------
  pdl_trigger();
  if (threadIdx.x == 0) {
    for (int i = 0; i < kAStages; ++i) {
      mbar_init(&s->a_full[i], 1);
      mbar_init(&s->a_empty[i], 1);               // the MMA commit
    }
    for (int i = 0; i < kQStages; ++i) {
      mbar_init(&s->q_full[i], 1);
      mbar_init(&s->q_empty[i], kDqGroupWarps);   // the dequant warps of the group that expanded it
    }
    for (int i = 0; i < kDqStages; ++i) {
      mbar_init(&s->dq_full[i], kDqGroupWarps);
      mbar_init(&s->dq_empty[i], 1);
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
    prefetch_tensormap(&tm_a);
  }
  if (warp == kMmaWarp) {
    tmem_alloc(&s->tmem_addr, kTmemCols);
    tmem_relinquish();
  }
  pdl_wait();  // nothing above read the predecessor's results
  build_tile_list(s->off, s->prefix, p.offsets, p.rows_total, p.E, C::kRows, p.n_tiles);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = s->tmem_addr;
  const int total_tiles = s->prefix[p.E];
  const int num_ctas = balanced_cta_count(total_tiles, gridDim.x);
  const int first_tile = static_cast<int>(blockIdx.x) < num_ctas ? static_cast<int>(blockIdx.x) : total_tiles;
  const int KS = p.ksteps;

  // weight rows (within the [E*N] row space) of a tile's two halves
  auto b_rows = [&](const TileCoord& c, int& n_lo, int& n_hi) {
    if (MODE == kModeGateUp) {
      n_lo = c.n_tile * BNH;
      n_hi = n_lo + p.I;
    } else {
      n_lo = c.n_tile * BN;
      n_hi = n_lo + BNH;
    }
  };

  if (warp == kTmaWarp) {
    // =============================== TMA producer =====================================
    if (lane == 0) {
      int as = 0, qs = 0;
      uint32_t a_phase = 0, q_phase = 0;
      uint32_t a_armed = 0, a_armed_parity = 0, q_armed = 0, q_armed_parity = 0;
      int cur_e = 0;
      bool ok = true;
      for (int T = first_tile; ok && T < total_tiles; T += num_ctas) {
        const TileCoord c = decode_tile(s->off, s->prefix, C::kRows, T, cur_e);
        int n_lo, n_hi;
        b_rows(c, n_lo, n_hi);
        const int NB = p.N / BNH;  // 128-row blocks per expert; a half tile past N re-reads the last one
        const uint8_t* q_lo = p.b_packed + (static_cast<int64_t>(c.e) * NB + n_lo / BNH) * KS * kQHalfBytes;
        const uint8_t* q_hi = p.b_packed + (static_cast<int64_t>(c.e) * NB + min(n_hi / BNH, NB - 1)) * KS * kQHalfBytes;
        for (int ks = 0; ks < KS; ++ks) {
          // codes first: their ring frees as soon as they are in registers, and for decode-sized
          // calls they are the stream from HBM that has to run ahead
          if (!wait_or_abort(&s->q_empty[qs], q_phase ^ 1, s, p)) { ok = false; break; }
          uint8_t* q_dst = q_base + static_cast<size_t>(qs) * kQBytes;
          mbar_arrive_expect_tx(&s->q_full[qs], kQBytes);
          bulk_load_1d(q_dst, q_lo + static_cast<int64_t>(ks) * kQHalfBytes, kQHalfBytes, &s->q_full[qs]);
          bulk_load_1d(q_dst + kQHalfBytes, q_hi + static_cast<int64_t>(ks) * kQHalfBytes, kQHalfBytes, &s->q_full[qs]);
          q_armed |= 1u << qs;
          q_armed_parity = (q_armed_parity & ~(1u << qs)) | (q_phase << qs);
          if (++qs == kQStages) { qs = 0; q_phase ^= 1; }

          if (!wait_or_abort(&s->a_empty[as], a_phase ^ 1, s, p)) { ok = false; break; }
          uint8_t* a_dst = smem + static_cast<size_t>(as) * kABytes;
          mbar_arrive_expect_tx(&s->a_full[as], kABytes);
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
            tma_load_2d(a_dst + mt * kAHalfBytes, &tm_a, &s->a_full[as], ks * BK, c.m0 + mt * BM);
          a_armed |= 1u << as;
          a_armed_parity = (a_armed_parity & ~(1u << as)) | (a_phase << as);
          if (++as == kAStages) { as = 0; a_phase ^= 1; }
        }
      }
      if (!ok) {  // let copies in flight land before the CTA's shared memory is released
        for (int i = 0; i < kAStages; ++i)
          if (a_armed & (1u << i)) mbar_wait_bounded(&s->a_full[i], (a_armed_parity >> i) & 1u, 20000000ull);
        for (int i = 0; i < kQStages; ++i)
          if (q_armed & (1u << i)) mbar_wait_bounded(&s->q_full[i], (q_armed_parity >> i) & 1u, 20000000ull);
      }
    }
  } else if (warp == kMmaWarp) {
    // =============================== MMA issuer =======================================
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16_f32(BM, BN);
      int ls = 0, ds = 0, acc = 0;
      uint32_t ld_phase = 0, dq_phase = 0, acc_phase = 0;
      bool ok = true;
      for (int T = first_tile; ok && T < total_tiles; T += num_ctas) {
        if (!wait_or_abort(&s->tmem_empty[acc], acc_phase ^ 1, s, p)) { ok = false; break; }
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * MT) * BN;
        for (int ks = 0; ks < KS; ++ks) {
          if (!wait_or_abort(&s->a_full[ls], ld_phase, s, p)) { ok = false; break; }
          if (!wait_or_abort(&s->dq_full[ds], dq_phase, s, p)) { ok = false; break; }
          tc_fence_after_sync();
          const uint64_t a_desc = umma_desc_k_sw128(smem_u32(smem + static_cast<size_t>(ls) * kABytes));
          const uint64_t b_desc = umma_desc_k_sw128(smem_u32(dq_base + static_cast<size_t>(ds) * kDqBytes));
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)  // the 128-row halves of A share the expanded weight tile
#pragma unroll
            for (int k4 = 0; k4 < BK / 16; ++k4)  // +32 bytes of K = +2 in the 16-byte address field
              umma_bf16(d_tmem + mt * BN, a_desc + mt * (kAHalfBytes >> 4) + 2 * k4, b_desc + 2 * k4, idesc,
                        (ks > 0 || k4 > 0) ? 1u : 0u);
          umma_commit(&s->a_empty[ls]);
          umma_commit(&s->dq_empty[ds]);
          if (ks == KS - 1) umma_commit(&s->tmem_full[acc]);
          if (++ls == kAStages) { ls = 0; ld_phase ^= 1; }
          if (++ds == kDqStages) { ds = 0; dq_phase ^= 1; }
        }
        if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1; }
      }
      // Nothing of this CTA's tensor work may be in flight when its TMEM and shared memory go
      // away: after an abort some MMAs may still be executing, so wait (bounded) for them.
      if (!ok) {
        umma_commit(&s->teardown);
        mbar_wait_bounded(&s->teardown, 0, 20000000ull);
      }
    }
  } else if (warp >= kEpiWarps && warp < kEpiWarps + kDqWarps) {
    // =============================== dequantization warps =============================
    // Two groups of 8 warps take alternate K-steps (a tile has an even number of them), so the
    // latency of one step's loads, barrier waits and stores hides behind the other group's math.
    const int grp = (warp - kEpiWarps) / kDqGroupWarps;
    const int n = ((warp - kEpiWarps) % kDqGroupWarps) * 32 + lane;  // weight row of the tile, 0..255
    const int half = n >> 7, nr = n & 127;
    const int KG = KS / 2;                         // 128-element groups along K: one K-step of each per group of warps
    uint32_t step0 = 0;                            // K-steps of this CTA before the current tile
    int cur_e = 0;
    bool ok = true;
    // (s, z) of group g of this thread's row in tile c; rows past N (dense, ragged N) clamp
    auto sz_index = [&](const TileCoord& c, int g) -> int64_t {
      int n_lo, n_hi;
      b_rows(c, n_lo, n_hi);
      const int row = min((half ? n_hi : n_lo) + nr, p.N - 1);
      return (static_cast<int64_t>(c.e) * KG + g) * p.N + row;
    };
    int T = first_tile;
    if (T < total_tiles) {
      TileCoord c = decode_tile(s->off, s->prefix, C::kRows, T, cur_e);
      int64_t idx = sz_index(c, 0);
      uint32_t s_next = __ldg(p.b_scales + idx), z_next = FMT == kFmtInt4 ? __ldg(p.b_zeros + idx) : 0u;
      for (;;) {
        const int Tn = T + num_ctas;
        const bool has_next = Tn < total_tiles;
        TileCoord cn = c;
        for (int g = 0; g < KG; ++g) {
          uint32_t s2, zc2;  // integer: s and 128 + z as bf16x2; e2m1: the two per-group factors
          if constexpr (FMT == kFmtInt4) {
            s2 = s_next | (s_next << 16);
            zc2 = (0x4300u | z_next) * 0x00010001u;
          } else {
            fp4_group_consts(s_next, zc2, s2);
          }
          if (g + 1 < KG) {
            idx = sz_index(c, g + 1);
          } else if (has_next) {
            cn = decode_tile(s->off, s->prefix, C::kRows, Tn, cur_e);
            idx = sz_index(cn, 0);
          }
          s_next = __ldg(p.b_scales + idx);
          if constexpr (FMT == kFmtInt4) z_next = __ldg(p.b_zeros + idx);
          const uint32_t step = step0 + 2 * g + grp;
          const uint32_t qs = step % kQStages, q_phase = (step / kQStages) & 1u;
          const uint32_t ds = step % kDqStages, dq_phase = (step / kDqStages) & 1u;
          if (!warp_wait_or_abort(&s->q_full[qs], q_phase, s, p)) { ok = false; break; }
          // a chunk is [word quad 0..1][row][16 bytes]: consecutive threads read consecutive pieces
          const uint4* q_src = reinterpret_cast<const uint4*>(q_base + static_cast<size_t>(qs) * kQBytes +
                                                              half * kQHalfBytes + nr * 16);
          const uint4 q0 = q_src[0], q1 = q_src[kQHalfBytes / 32];
          __syncwarp();
          if (lane == 0) mbar_arrive(&s->q_empty[qs]);  // the codes are in registers
          if (!warp_wait_or_abort(&s->dq_empty[ds], dq_phase ^ 1, s, p)) { ok = false; break; }
          uint8_t* row_dst = dq_base + static_cast<size_t>(ds) * kDqBytes + n * 128;
          const uint32_t words[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
          for (int i = 0; i < 8; ++i)  // 16-byte chunk i of the row lands at chunk i ^ (row % 8): SWIZZLE_128B
            *reinterpret_cast<uint4*>(row_dst + ((i ^ (n & 7)) << 4)) =
                FMT == kFmtInt4 ? dequant_word(words[i], zc2, s2) : dequant_word_fp4(words[i], zc2, s2);
          fence_proxy_async_smem();  // generic-proxy stores -> visible to the tensor core's async proxy
          __syncwarp();
          if (lane == 0) mbar_arrive(&s->dq_full[ds]);
        }
        if (!ok || !has_next) break;
        step0 += static_cast<uint32_t>(KS);
        T = Tn;
        c = cn;
      }
    }
  } else if (warp < kEpiWarps) {
    // =============================== epilogue warps ===================================
    const int q = warp;              // TMEM lane quadrant
    const int r = q * 32 + lane;     // row within the tile
    const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
    int acc = 0;
    uint32_t acc_phase = 0;
    int cur_e = 0;
    for (int T = first_tile; T < total_tiles; T += num_ctas) {
      const TileCoord c = decode_tile(s->off, s->prefix, C::kRows, T, cur_e);
      bool ok = true;
#pragma unroll 1
      for (int mt = 0; mt < MT; ++mt) {
      const int row = c.m0 + mt * BM + r;
      const bool valid = row < c.m_end;
      const bool warp_live = c.m0 + mt * BM + q * 32 < c.m_end;
      float w = 0.0f;
      int64_t out_row = row;
      if (MODE == kModeDown && valid) {
        w = __ldg(p.pair_weights + row);
        // no pair map: the contribution stays at its sorted position
        if (p.sorted_pair) out_row = min(max(__ldg(p.sorted_pair + row), 0), p.rows_total - 1);  // in bounds even after bad ids
      }
      if (mt == 0) {
        if (!warp_wait_or_abort(&s->tmem_full[acc], acc_phase, s, p)) { ok = false; break; }
        tc_fence_after_sync();
      }
      const uint32_t t0 = tmem_base + lane_addr + static_cast<uint32_t>((acc * MT + mt) * BN);
      if (warp_live) {
        if (MODE == kModeGateUp) {
#pragma unroll 1
          for (int ch = 0; ch < BNH / 16; ++ch) {
            uint32_t vg[16], vu[16];
            tmem_ld_x16(t0 + 16 * ch, vg);
            tmem_ld_x16(t0 + BNH + 16 * ch, vu);
            tmem_ld_wait();
            uint32_t gb[8], ub[8], hb[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              gb[j] = bf16x2_bits(__uint_as_float(vg[2 * j]), __uint_as_float(vg[2 * j + 1]));
              ub[j] = bf16x2_bits(__uint_as_float(vu[2 * j]), __uint_as_float(vu[2 * j + 1]));
              const float h0 = silu_mul(bf16_bits_to_f32(gb[j] & 0xFFFFu), bf16_bits_to_f32(ub[j] & 0xFFFFu));
              const float h1 = silu_mul(__uint_as_float(gb[j] & 0xFFFF0000u), __uint_as_float(ub[j] & 0xFFFF0000u));
              hb[j] = bf16x2_bits(h0, h1);
            }
            if (valid) {
              const int col = c.n_tile * BNH + 16 * ch;
              uint4* hd = reinterpret_cast<uint4*>(p.h_bf16 + static_cast<int64_t>(row) * p.I + col);
              hd[0] = make_uint4(hb[0], hb[1], hb[2], hb[3]);
              hd[1] = make_uint4(hb[4], hb[5], hb[6], hb[7]);
              if (p.out_bf16) {  // debug dump of the bf16 gate_up row
                uint4* gd = reinterpret_cast<uint4*>(p.out_bf16 + static_cast<int64_t>(row) * p.N + col);
                gd[0] = make_uint4(gb[0], gb[1], gb[2], gb[3]);
                gd[1] = make_uint4(gb[4], gb[5], gb[6], gb[7]);
                uint4* ud = reinterpret_cast<uint4*>(p.out_bf16 + static_cast<int64_t>(row) * p.N + p.I + col);
                ud[0] = make_uint4(ub[0], ub[1], ub[2], ub[3]);
                ud[1] = make_uint4(ub[4], ub[5], ub[6], ub[7]);
              }
            }
          }
        } else {
#pragma unroll 1
          for (int ch = 0; ch < BN / 16; ++ch) {
            uint32_t v[16];
            tmem_ld_x16(t0 + 16 * ch, v);
            tmem_ld_wait();
            const int col = c.n_tile * BN + 16 * ch;
            if (valid && col < p.N) {
              if (p.out_f32) {  // fp32 accumulator dump (down: in sorted order)
                float4* fd = reinterpret_cast<float4*>(p.out_f32 + static_cast<int64_t>(row) * p.N + col);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                  fd[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                      __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
              }
              uint32_t ob[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                float a = __uint_as_float(v[2 * j]), b = __uint_as_float(v[2 * j + 1]);
                if (MODE == kModeDown) {  // contribution = bf16( fl(w * y) )
                  a = __fmul_rn(w, a);
                  b = __fmul_rn(w, b);
                }
                ob[j] = bf16x2_bits(a, b);
              }
              if (p.out_bf16) {
                uint4* od = reinterpret_cast<uint4*>(p.out_bf16 + out_row * p.N + col);
                od[0] = make_uint4(ob[0], ob[1], ob[2], ob[3]);
                od[1] = make_uint4(ob[4], ob[5], ob[6], ob[7]);
              }
            }
          }
        }
      }
      }  // mt
      if (!ok) break;
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&s->tmem_empty[acc]);
      if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1; }
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

CUresult make_tmap_a(EncodeTiledFn encode, CUtensorMap* m, const void* base, uint64_t rows, uint64_t K) {
  // bf16 tensor [rows, K] row-major; box = 64 elements (128 bytes) x 128 rows, 128-byte swizzle.
  const cuuint64_t dims[2] = {K, rows};
  const cuuint64_t strides[1] = {K * 2};
  const cuuint32_t box[2] = {BK, BM};
  const cuuint32_t estr[2] = {1, 1};
  return encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

template <int MODE, int MT, int FMT>
cudaError_t launch_mode(const Launch& L, const CUtensorMap& ta, const W4Params& p, const GemmW4Args& a) {
  // sticky per function and device; atomic: contexts on several host threads may launch at once (both
  // would set the same value)
  static std::atomic<bool> attr_set_dev[64];
  std::atomic<bool>& attr_set = attr_set_dev[L.device & 63];
  if (!attr_set.load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_w4a16_kernel<MODE, MT, FMT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem_bytes<MT>()));
    if (e != cudaSuccess) return e;
    attr_set.store(true, std::memory_order_release);
  }
  // upper bound on the tile count (group sizes live on the device): each expert adds at most
  // one partial row tile
  const int64_t m_tiles_max = a.rows_total / Cfg<MT>::kRows + a.E;
  const int grid = static_cast<int>(std::min<int64_t>(L.sm_count, m_tiles_max * p.n_tiles));
  ++*L.launches;
  return launch_pdl(gemm_w4a16_kernel<MODE, MT, FMT>, static_cast<unsigned>(grid), kThreads, smem_bytes<MT>(), L.stream,
                    ta, p);
}

template <int MODE, int FMT>
cudaError_t launch_fmt(const Launch& L, const CUtensorMap& ta, const W4Params& p, const GemmW4Args& a) {
  // groups of at most 128 rows on average (decode-sized calls): 128-row tiles
  if (a.rows_total <= a.E * BM) return launch_mode<MODE, 1, FMT>(L, ta, p, a);
  return launch_mode<MODE, 2, FMT>(L, ta, p, a);
}

template <int MODE>
cudaError_t launch_mt(const Launch& L, const CUtensorMap& ta, const W4Params& p, const GemmW4Args& a) {
  return a.fmt == kFmtE2m1 ? launch_fmt<MODE, kFmtE2m1>(L, ta, p, a) : launch_fmt<MODE, kFmtInt4>(L, ta, p, a);
}

}  // namespace

cudaError_t launch_gemm_w4a16(const Launch& L, EncodeTiledFn encode, const GemmW4Args& a, CUresult* cu_err) {
  *cu_err = CUDA_SUCCESS;
  if (a.rows_total == 0) return cudaSuccess;
  // decode-sized groups: the swapped-operand kernel (bitwise the same rows, far less expansion work per token)
  if (L.gemm_path == 2 ? a.offsets != nullptr : (L.gemm_path == 0 && gemm_w4a16_decode_applies(a)))
    return launch_gemm_w4a16_decode(L, encode, a, cu_err);
  CUtensorMap ta;
  CUresult r = make_tmap_a(encode, &ta, a.a_bf16, static_cast<uint64_t>(a.rows_total), static_cast<uint64_t>(a.K));
  if (r != CUDA_SUCCESS) {
    *cu_err = r;
    return cudaErrorUnknown;
  }
  W4Params p{};
  p.b_packed = a.b_packed;
  p.b_scales = a.b_scales;
  p.b_zeros = a.b_zeros;
  p.offsets = a.offsets;
  p.rows_total = static_cast<int>(a.rows_total);
  p.ksteps = static_cast<int>(a.K / BK);
  p.N = static_cast<int>(a.N);
  p.E = static_cast<int>(a.E);
  p.I = static_cast<int>(a.N / 2);
  p.n_tiles = a.mode == kModeGateUp ? static_cast<int>(a.N / 2 / BNH) : static_cast<int>((a.N + BN - 1) / BN);
  p.out_bf16 = a.out_bf16;
  p.out_f32 = a.out_f32;
  p.h_bf16 = a.h_bf16;
  p.sorted_pair = a.sorted_pair;
  p.pair_weights = a.pair_weights;
  p.status = L.d_status;
  p.wait_limit_ns = 2000000000ull;
  switch (a.mode) {
    case kModeLinear: return launch_mt<kModeLinear>(L, ta, p, a);
    case kModeGateUp: return launch_mt<kModeGateUp>(L, ta, p, a);
    case kModeDown: return launch_mt<kModeDown>(L, ta, p, a);
  }
  return cudaErrorInvalidValue;
}

}  // namespace qarl
