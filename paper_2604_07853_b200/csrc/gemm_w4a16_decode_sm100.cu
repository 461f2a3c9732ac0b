// W4A16 grouped GEMM for decode-sized row groups (a few tokens per expert): the arithmetic of
// gemm_w4a16_sm100.cu with the operands of the MMA swapped.
//
//   y[t, n] = sum_k x[t, k] * w^[n, k],   w^ = bf16( s * (W_q - z) )   (Dequant of Sec. 2.2)
//
// With ~16 rows per expert the wide kernel expands 256 weight rows per K-step for a token tile that
// is almost empty: 32 KB of shared-memory stores and a 128 x 256 x 16 MMA on padding, which made the
// 4-bit layer slower at decode than the FP8 one although it streams half the bytes (Appendix D.1:
// decode is memory-bound, so the narrower format should win).  Here the 128 expanded WEIGHT rows of a
// block are the M side of tcgen05.mma and at most 32 TOKEN rows its N side:
//   D[n, t] = sum_k w^[n, k] x[t, k]      (kind::f16, M = 128, N = 32, K = 16, four per 64-element K-step)
// The bf16 products are exact and the instruction adds them in the same order whichever operand
// carries which matrix (checked bit for bit on the device: 10^8 random bf16 dot products, N = 16 ...
// 128), and the whole K reduction accumulates in TMEM in ascending k in both kernels, so a token's
// output row has the same bits here and in the wide kernel (the tile-size invariance tests compare).
//
// A tile = (expert e, pair of weight blocks j, chunk of <= 32 rows of the expert's group):
//   gate_up: blocks j (gate rows) and j + I/128 (the matching up rows); down/linear: blocks 2j, 2j+1.
// A stage is one 128-element quantization group of K (two K-steps of 64): what bounds a kernel of this
// shape is the fixed cost per stage of the single threads that wait, issue and commit, so stages are as
// large as shared memory allows and every such thread has one job.
// CTA = 768 threads: warps 0-3 epilogue (thread = weight row: TMEM -> SwiGLU / weighting -> bf16,
// transposed through shared memory so that global stores are whole token rows), warps 4-11 / 12-19
// dequantization of the tile's first / second weight block (two threads per weight row; they read
// their codes straight from global memory, three stages ahead, into registers), warp 21 producer of
// the token rows (TMA), warps 22 / 23 MMA issuers of the two blocks (warp 20 only starts the CTA's
// first tile's codes towards L2 while the kernel still waits for its predecessor).
// Every barrier wait is bounded; an expired wait aborts the CTA cleanly.
#include <algorithm>
#include <atomic>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "sched.cuh"
#include "w4_dequant.cuh"

namespace qarl {
namespace {

using namespace ptx;

constexpr int BW = 128;            // weight rows per block (UMMA M)
constexpr int NT = 32;             // token rows per tile (UMMA N)
constexpr int BK = 64;             // bf16 elements per K-step (128 bytes)
constexpr int kGK = 2;             // K-steps per stage: one 128-element quantization group
constexpr int kEpiWarps = 4;       // warps 0-3
constexpr int kDqHalfWarps = 8;    // warps 4-11 expand the tile's first block, warps 12-19 its second
constexpr int kCodeWarp = 20;      // producer of the codes
constexpr int kTokenWarp = 21;     // producer of the token rows
constexpr int kMmaWarp0 = 22;      // MMA issuer of the first block (warp 23: of the second)
constexpr int kThreads = 24 * 32;
constexpr uint32_t kQStepBytes = BW * BK / 2;            // 4 KB: 128 rows x 32 bytes of codes (one K-step of one block)
constexpr uint32_t kQHalfBytes = kGK * kQStepBytes;      // 8 KB: one block, one group
constexpr uint32_t kXStepBytes = NT * BK * 2;            // 4 KB: 32 token rows x 64 bf16
constexpr uint32_t kXBytes = kGK * kXStepBytes;          // 8 KB per stage
constexpr uint32_t kDqStepBytes = BW * BK * 2;           // 16 KB: one expanded block, one K-step
constexpr uint32_t kDqBytes = kGK * kDqStepBytes;        // 32 KB per stage and block
constexpr int kCodeAhead = 3;       // stages whose codes a dequantization thread holds in registers ahead of use
constexpr int kXStages = 4;
constexpr int kDqStages = 2;       // per block
constexpr int kAccBufs = 4;        // TMEM accumulators of 2 x NT columns
constexpr uint32_t kTmemCols = 256;
constexpr int kMaxExperts = 1024;
constexpr int kOutRowBytes = 2 * BW * 2 + 16;    // bf16 row of 256 outputs, padded
constexpr uint32_t kOutBytes = NT * kOutRowBytes;
constexpr uint32_t kPrefetchChunk = 32768;       // bytes per L2 prefetch instruction

struct W4DecodeParams {
  const uint8_t* b_packed;   // tile-major 4 KB chunks [E][N/128][K/64]
  const uint16_t* b_scales;  // bf16 bits [E][K/128][N]
  const uint8_t* b_zeros;    // [E][K/128][N]
  const int32_t* offsets;
  int rows_total;
  int ksteps;                // K / 64
  int N;
  int E;
  int n_pairs;
  int I;
  uint16_t* out_bf16;        // linear: y; down: contributions; gate_up (debug): bf16 gate_up
  float* out_f32;
  uint16_t* h_bf16;
  const int32_t* sorted_pair;
  const float* pair_weights;
  int* status;
  unsigned long long wait_limit_ns;
};

struct __align__(8) SmemTail {
  uint64_t x_full[kXStages];
  uint64_t x_empty[kXStages];
  uint64_t dq_full[2][kDqStages];
  uint64_t dq_empty[2][kDqStages];
  uint64_t tmem_full[kAccBufs];
  uint64_t tmem_empty[kAccBufs];
  uint64_t teardown[2];
  uint32_t tmem_addr;
  int abort_flag;
  int32_t off[kMaxExperts + 1];
  int32_t prefix[kMaxExperts + 1];
};

constexpr size_t kSmemBytes = 1024 + static_cast<size_t>(kXStages) * kXBytes +
                              2 * static_cast<size_t>(kDqStages) * kDqBytes + kOutBytes + sizeof(SmemTail);
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, SmemTail* s, const W4DecodeParams& p) {
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
// whole warp: every lane polls, then the lanes vote (no split warp after a wait; one polling lane
// with the others parked at a shuffle measured 30 % slower here)
__device__ __forceinline__ bool warp_wait_or_abort(uint64_t* bar, uint32_t parity, SmemTail* s, const W4DecodeParams& p) {
  return __all_sync(0xFFFFFFFFu, wait_or_abort(bar, parity, s, p) ? 1 : 0) != 0;
}

// Barrier among `n` threads that also tells every one of them whether `pred` held for all.
__device__ __forceinline__ bool named_bar_all(uint32_t id, uint32_t n, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t"
      ".reg .pred p, q;\n\t"
      "setp.ne.b32 q, %3, 0;\n\t"
      "bar.red.and.pred p, %1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t"
      "}"
      : "=r"(r)
      : "r"(id), "r"(n), "r"(static_cast<uint32_t>(pred))
      : "memory");
  return r != 0;
}

__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

// 128-row blocks (within the expert) of a tile's two halves
template <int MODE>
__device__ __forceinline__ void tile_blocks(const W4DecodeParams& p, int j, int& nb_lo, int& nb_hi) {
  const int NB = p.N / BW;
  if (MODE == kModeGateUp) {
    nb_lo = j;
    nb_hi = j + p.I / BW;
  } else {
    nb_lo = 2 * j;
    nb_hi = min(2 * j + 1, NB - 1);  // a half past N re-reads the last block; its columns are never stored
  }
}

template <int MODE, int FMT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_w4a16_decode_kernel(const __grid_constant__ CUtensorMap tm_x, const W4DecodeParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* dq_base = smem;                                                   // [block][stage][K-step][16 KB], 1024-byte aligned
  uint8_t* x_base = dq_base + 2 * static_cast<size_t>(kDqStages) * kDqBytes;  // [stage][K-step][4 KB]
  uint8_t* out_tile = x_base + static_cast<size_t>(kXStages) * kXBytes;
  SmemTail* s = reinterpret_cast<SmemTail*>(out_tile + kOutBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- set-up: barriers, TMEM, tile list ------------------------------------------------
  pdl_trigger();
  if (threadIdx.x == 0) {
    for (int i = 0; i < kXStages; ++i) {
      mbar_init(&s->x_full[i], 1);
      mbar_init(&s->x_empty[i], 2);               // the commits of the two MMA issuers
    }
    for (int h = 0; h < 2; ++h)
      for (int i = 0; i < kDqStages; ++i) {
        mbar_init(&s->dq_full[h][i], kDqHalfWarps);
        mbar_init(&s->dq_empty[h][i], 1);
      }
    for (int i = 0; i < kAccBufs; ++i) {
      mbar_init(&s->tmem_full[i], 2);
      mbar_init(&s->tmem_empty[i], kEpiWarps);
    }
    mbar_init(&s->teardown[0], 1);
    mbar_init(&s->teardown[1], 1);
    s->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kTokenWarp && lane == 0) prefetch_tensormap(&tm_x);
  if (warp == kMmaWarp0) {
    tmem_alloc(&s->tmem_addr, kTmemCols);
    tmem_relinquish();
  }
  const int KS = p.ksteps;
  const int KG = KS / kGK;           // 128-element groups along K
  const int NB = p.N / BW;
  // codes of tile (expert e, block pair j): the two blocks' chunks, each KS x 4 KB contiguous
  auto tile_codes = [&](int e, int j, const uint8_t*& q_lo, const uint8_t*& q_hi) {
    int nb_lo, nb_hi;
    tile_blocks<MODE>(p, j, nb_lo, nb_hi);
    q_lo = p.b_packed + (static_cast<int64_t>(e) * NB + nb_lo) * KS * kQStepBytes;
    q_hi = p.b_packed + (static_cast<int64_t>(e) * NB + nb_hi) * KS * kQStepBytes;
  };
  // pull a whole tile's codes towards L2 (used once, for the CTA's first tile, before the dependency wait)
  auto prefetch_tile = [&](int e, int j) {
    const uint8_t *q_lo, *q_hi;
    tile_codes(e, j, q_lo, q_hi);
    const uint32_t bytes = static_cast<uint32_t>(KS) * kQStepBytes;
    for (uint32_t o = 0; o < bytes; o += kPrefetchChunk) {
      bulk_prefetch_l2(q_lo + o, min(kPrefetchChunk, bytes - o));
      bulk_prefetch_l2(q_hi + o, min(kPrefetchChunk, bytes - o));
    }
  };
  if (warp == kCodeWarp && lane == 0) {
    // The weights do not depend on the kernels before this one in the stream: start pulling this CTA's
    // first tile (guessed as expert T / n_pairs, pair T % n_pairs: exact when every expert has one chunk).
    const int T = blockIdx.x;
    if (T < p.E * p.n_pairs) prefetch_tile(T / p.n_pairs, T % p.n_pairs);
  }
  pdl_wait();  // nothing above read the predecessor's results
  build_tile_list(s->off, s->prefix, p.offsets, p.rows_total, p.E, NT, p.n_pairs);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = s->tmem_addr;
  const int total_tiles = s->prefix[p.E];
  const int num_ctas = gridDim.x;
  const int first_tile = blockIdx.x;

  if (warp == kCodeWarp) {
    // (this warp only started the first tile's codes on their way to L2, above)
  } else if (warp == kTokenWarp) {
    // =============================== producer of the token rows =======================
    if (lane == 0) {
      int xs = 0, cur_e = 0;
      uint32_t x_phase = 0, x_armed = 0, x_armed_parity = 0;
      bool ok = true;
      for (int T = first_tile; ok && T < total_tiles; T += num_ctas) {
        const TileCoord c = decode_tile(s->off, s->prefix, NT, T, cur_e);
        for (int g = 0; g < KG; ++g) {
          if (!wait_or_abort(&s->x_empty[xs], x_phase ^ 1, s, p)) { ok = false; break; }
          mbar_arrive_expect_tx(&s->x_full[xs], kXBytes);
#pragma unroll
          for (int u = 0; u < kGK; ++u)
            tma_load_2d(x_base + static_cast<size_t>(xs) * kXBytes + u * kXStepBytes, &tm_x, &s->x_full[xs],
                        (g * kGK + u) * BK, c.m0);
          x_armed |= 1u << xs;
          x_armed_parity = (x_armed_parity & ~(1u << xs)) | (x_phase << xs);
          if (++xs == kXStages) { xs = 0; x_phase ^= 1; }
        }
      }
      if (!ok) {
        for (int i = 0; i < kXStages; ++i)
          if (x_armed & (1u << i)) mbar_wait_bounded(&s->x_full[i], (x_armed_parity >> i) & 1u, 20000000ull);
      }
    }
  } else if (warp >= kMmaWarp0) {
    // =============================== MMA issuers ======================================
    // One thread per weight block: each feeds its own 32 TMEM columns in ascending k, so the two never
    // touch the same accumulator, and the per-stage cost of waiting, issuing and committing is shared.
    if (lane == 0) {
      const int h = warp - kMmaWarp0;
      constexpr uint32_t idesc = umma_idesc_bf16_f32(BW, NT);
      int xs = 0, ds = 0, acc = 0;
      uint32_t x_phase = 0, dq_phase = 0, acc_phase = 0;
      bool ok = true;
      for (int T = first_tile; ok && T < total_tiles; T += num_ctas) {
        if (!wait_or_abort(&s->tmem_empty[acc], acc_phase ^ 1, s, p)) { ok = false; break; }
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc) * (2 * NT) + static_cast<uint32_t>(h) * NT;
        for (int g = 0; g < KG; ++g) {
          if (!wait_or_abort(&s->x_full[xs], x_phase, s, p)) { ok = false; break; }
          if (!wait_or_abort(&s->dq_full[h][ds], dq_phase, s, p)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t w_addr = smem_u32(dq_base + (static_cast<size_t>(h) * kDqStages + ds) * kDqBytes);
          const uint32_t x_addr = smem_u32(x_base + static_cast<size_t>(xs) * kXBytes);
#pragma unroll
          for (int u = 0; u < kGK; ++u) {
            const uint64_t w_desc = umma_desc_k_sw128(w_addr + u * kDqStepBytes);
            const uint64_t x_desc = umma_desc_k_sw128(x_addr + u * kXStepBytes);
#pragma unroll
            for (int k4 = 0; k4 < BK / 16; ++k4)  // +32 bytes of K = +2 in the 16-byte address field
              umma_bf16(d_tmem, w_desc + 2 * k4, x_desc + 2 * k4, idesc, (g > 0 || u > 0 || k4 > 0) ? 1u : 0u);
          }
          umma_commit(&s->dq_empty[h][ds]);
          umma_commit(&s->x_empty[xs]);
          if (g == KG - 1) umma_commit(&s->tmem_full[acc]);
          if (++xs == kXStages) { xs = 0; x_phase ^= 1; }
          if (++ds == kDqStages) { ds = 0; dq_phase ^= 1; }
        }
        if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1; }
      }
      if (!ok) {  // after an abort MMAs may still be executing: wait (bounded) before TMEM goes away
        umma_commit(&s->teardown[h]);
        mbar_wait_bounded(&s->teardown[h], 0, 20000000ull);
      }
    }
  } else if (warp >= kEpiWarps) {
    // =============================== dequantization warps =============================
    // Eight warps per weight block; two threads per weight row, one per K-step of the stage: 64 codes
    // each, one (s, z) for both (a stage is exactly one quantization group of the row).
    const int h = (warp - kEpiWarps) / kDqHalfWarps;
    const int idx = ((warp - kEpiWarps) % kDqHalfWarps) * 32 + lane;  // 0..255
    const int nr = idx & 127, u = idx >> 7;        // weight row of the block, K-step of the stage
    uint32_t stage = 0;                            // stages of this CTA so far
    int cur_e = 0;
    bool ok = true;
    // (s, z) of group g of this thread's row in tile c; rows past N (dense, ragged N) clamp
    auto sz_index = [&](const TileCoord& c, int g) -> int64_t {
      int nb_lo, nb_hi;
      tile_blocks<MODE>(p, c.n_tile, nb_lo, nb_hi);
      const int row = min((h ? nb_hi : nb_lo) * BW + nr, p.N - 1);
      return (static_cast<int64_t>(c.e) * KG + g) * p.N + row;
    };
    // The codes come straight from global memory, three stages ahead of their use, in registers: no
    // shared-memory ring and no hand-off between a producer thread and these warps stands between the
    // memory and the expansion.  Consecutive threads read consecutive 16-byte pieces of a 4 KB chunk
    // ([word quad 0..1][row][16 bytes]); the data are read once (streaming loads).  (Pulling a tile's codes
    // into L2 a tile ahead as well was measured and costs 7 % here.)
    int pfT = first_tile, pfg = 0, pf_e = 0;
    const uint8_t* pf_base = nullptr;  // this thread's piece of group 0 of tile pfT
    auto pf_set_tile = [&]() {
      if (pfT < total_tiles) {
        const TileCoord t = decode_tile(s->off, s->prefix, NT, pfT, pf_e);
        const uint8_t *q_lo, *q_hi;
        tile_codes(t.e, t.n_tile, q_lo, q_hi);
        pf_base = (h ? q_hi : q_lo) + u * kQStepBytes + nr * 16;
      }
    };
    auto pf_load = [&](uint4& a, uint4& b) {
      if (pfT < total_tiles) {
        const uint4* src = reinterpret_cast<const uint4*>(pf_base + static_cast<int64_t>(pfg) * kQHalfBytes);
        a = __ldcs(src);
        b = __ldcs(src + kQStepBytes / 32);
        if (++pfg == KG) {
          pfg = 0;
          pfT += num_ctas;
          pf_set_tile();
        }
      }
    };
    uint4 qa0 = make_uint4(0, 0, 0, 0), qa1 = qa0, qb0 = qa0, qb1 = qa0, qc0 = qa0, qc1 = qa0;
    static_assert(kCodeAhead == 3, "three register sets");
    pf_set_tile();
    pf_load(qa0, qa1);
    pf_load(qb0, qb1);
    pf_load(qc0, qc1);
    int T = first_tile;
    if (T < total_tiles) {
      TileCoord c = decode_tile(s->off, s->prefix, NT, T, cur_e);
      int64_t sz = sz_index(c, 0);
      uint32_t s_next = __ldg(p.b_scales + sz), z_next = FMT == kFmtInt4 ? __ldg(p.b_zeros + sz) : 0u;
      for (;;) {
        const int Tn = T + num_ctas;
        const bool has_next = Tn < total_tiles;
        TileCoord cn = c;
        for (int g = 0; g < KG; ++g, ++stage) {
          uint32_t s2, zc2;  // integer: s and 128 + z as bf16x2; e2m1: the two per-group factors
          if constexpr (FMT == kFmtInt4) {
            s2 = s_next | (s_next << 16);
            zc2 = (0x4300u | z_next) * 0x00010001u;
          } else {
            fp4_group_consts(s_next, zc2, s2);
          }
          if (g + 1 < KG) {
            sz = sz_index(c, g + 1);
          } else if (has_next) {
            cn = decode_tile(s->off, s->prefix, NT, Tn, cur_e);
            sz = sz_index(cn, 0);
          }
          s_next = __ldg(p.b_scales + sz);
          if constexpr (FMT == kFmtInt4) z_next = __ldg(p.b_zeros + sz);
          const uint32_t ds = stage % kDqStages, dq_phase = (stage / kDqStages) & 1u;
          const uint4 q0 = qa0, q1 = qa1;  // this stage's codes; the sets move up and the third one is refilled
          qa0 = qb0;
          qa1 = qb1;
          qb0 = qc0;
          qb1 = qc1;
          pf_load(qc0, qc1);
          if (!warp_wait_or_abort(&s->dq_empty[h][ds], dq_phase ^ 1, s, p)) { ok = false; break; }
          uint8_t* row_dst = dq_base + (static_cast<size_t>(h) * kDqStages + ds) * kDqBytes + u * kDqStepBytes + nr * 128;
          const uint32_t words[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
          for (int i = 0; i < 8; ++i)  // 16-byte chunk i of the row lands at chunk i ^ (row % 8): SWIZZLE_128B
            *reinterpret_cast<uint4*>(row_dst + ((i ^ (nr & 7)) << 4)) =
                FMT == kFmtInt4 ? dequant_word(words[i], zc2, s2) : dequant_word_fp4(words[i], zc2, s2);
          fence_proxy_async_smem();  // generic-proxy stores -> visible to the tensor core's async proxy
          __syncwarp();
          if (lane == 0) mbar_arrive(&s->dq_full[h][ds]);
        }
        if (!ok || !has_next) break;
        T = Tn;
        c = cn;
      }
    }
  } else {
    // =============================== epilogue warps ===================================
    const int wr = warp * 32 + lane;  // weight row within a block = TMEM lane
    constexpr uint32_t kEpiThreads = kEpiWarps * 32;
    const uint32_t lane_addr = static_cast<uint32_t>(warp * 32) << 16;
    int acc = 0, cur_e = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    uint16_t* T16 = reinterpret_cast<uint16_t*>(out_tile);
    for (int T = first_tile; T < total_tiles; T += num_ctas) {
      const TileCoord c = decode_tile(s->off, s->prefix, NT, T, cur_e);
      const int rows = min(NT, c.m_end - c.m0);  // live token rows of this tile (>= 1)
      const int j = c.n_tile;
      ok = warp_wait_or_abort(&s->tmem_full[acc], acc_phase, s, p);
      ok = named_bar_all(1, kEpiThreads, ok);  // one decision for the four warps; the previous tile's row readers are done
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t t0 = tmem_base + lane_addr + static_cast<uint32_t>(acc) * (2 * NT);
      const int col_lo = 2 * j * BW + wr, col_hi = col_lo + BW;  // down / linear: this thread's two output columns
      const bool hi_ok = col_hi < p.N;
      // 16 token columns at a time (the register budget of a 704-thread CTA)
#pragma unroll 1
      for (int tc = 0; tc < NT; tc += 16) {
        uint32_t vl[16], vh[16];
        tmem_ld_x16(t0 + tc, vl);
        tmem_ld_x16(t0 + NT + tc, vh);
        tmem_ld_wait();
        if (tc + 16 == NT) {  // the accumulator is in registers: hand it back
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&s->tmem_empty[acc]);
        }
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          const int t = tc + u;
          if (MODE == kModeGateUp) {
            // h = bf16( silu(bf16 gate) * bf16 up ), this thread's column of the tile's 128 h columns
            const uint32_t gb = f32_to_bf16_bits(__uint_as_float(vl[u])), ub = f32_to_bf16_bits(__uint_as_float(vh[u]));
            const uint32_t hb = f32_to_bf16_bits(silu_mul(bf16_bits_to_f32(gb), bf16_bits_to_f32(ub)));
            T16[t * (kOutRowBytes / 2) + wr] = static_cast<uint16_t>(hb);
            if (p.out_bf16 && t < rows) {  // debug dump of the bf16 gate_up row
              uint16_t* gd = p.out_bf16 + static_cast<int64_t>(c.m0 + t) * p.N + j * BW + wr;
              gd[0] = static_cast<uint16_t>(gb);
              gd[p.I] = static_cast<uint16_t>(ub);
            }
          } else {
            float lo = __uint_as_float(vl[u]), hi = __uint_as_float(vh[u]);
            if (p.out_f32 && t < rows) {  // fp32 accumulator dump (down: in sorted order)
              float* d = p.out_f32 + static_cast<int64_t>(c.m0 + t) * p.N;
              d[col_lo] = lo;
              if (hi_ok) d[col_hi] = hi;
            }
            if (MODE == kModeDown) {  // contribution = bf16( fl(w * y) )
              const float w = __ldg(p.pair_weights + min(c.m0 + t, p.rows_total - 1));
              lo = __fmul_rn(w, lo);
              hi = __fmul_rn(w, hi);
            }
            T16[t * (kOutRowBytes / 2) + wr] = static_cast<uint16_t>(f32_to_bf16_bits(lo));
            T16[t * (kOutRowBytes / 2) + BW + wr] = static_cast<uint16_t>(f32_to_bf16_bits(hi));
          }
        }
      }
      if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1; }

      if (MODE == kModeGateUp) {
        named_bar_sync(2, kEpiThreads);
        for (int t = warp; t < rows; t += kEpiWarps) {  // a warp per token row: 256 bytes, 8 per lane
          const uint2 hv = *reinterpret_cast<const uint2*>(out_tile + t * kOutRowBytes + lane * 8);
          *reinterpret_cast<uint2*>(p.h_bf16 + static_cast<int64_t>(c.m0 + t) * p.I + j * BW + lane * 4) = hv;
        }
      } else {
        named_bar_sync(2, kEpiThreads);
        if (p.out_bf16) {
          for (int t = warp; t < rows; t += kEpiWarps) {  // a warp per output row: 512 bytes, 16 per lane
            const int row = c.m0 + t;
            int64_t out_row = row;
            if (MODE == kModeDown && p.sorted_pair) out_row = min(max(__ldg(p.sorted_pair + row), 0), p.rows_total - 1);
            const uint4 v = *reinterpret_cast<const uint4*>(out_tile + t * kOutRowBytes + lane * 16);
            const int col = 2 * j * BW + 8 * lane;
            if (col < p.N) *reinterpret_cast<uint4*>(p.out_bf16 + out_row * p.N + col) = v;
          }
        }
      }
    }
  }

  // ---- teardown ---------------------------------------------------------------------------
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

CUresult make_tmap_x(EncodeTiledFn encode, CUtensorMap* m, const void* base, uint64_t rows, uint64_t K) {
  // bf16 tensor [rows, K] row-major; box = 64 elements (128 bytes) x 32 rows, 128-byte swizzle.
  const cuuint64_t dims[2] = {K, rows};
  const cuuint64_t strides[1] = {K * 2};
  const cuuint32_t box[2] = {BK, NT};
  const cuuint32_t estr[2] = {1, 1};
  return encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

template <int MODE, int FMT>
cudaError_t launch_mode(const Launch& L, const CUtensorMap& tx, const W4DecodeParams& p, int grid) {
  static std::atomic<bool> attr_set_dev[64];  // sticky per function and device; set idempotently
  std::atomic<bool>& attr_set = attr_set_dev[L.device & 63];
  if (!attr_set.load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_w4a16_decode_kernel<MODE, FMT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kSmemBytes));
    if (e != cudaSuccess) return e;
    attr_set.store(true, std::memory_order_release);
  }
  ++*L.launches;
  return launch_pdl(gemm_w4a16_decode_kernel<MODE, FMT>, static_cast<unsigned>(grid), kThreads, kSmemBytes, L.stream, tx, p);
}

template <int MODE>
cudaError_t launch_fmt(const Launch& L, const CUtensorMap& tx, const W4DecodeParams& p, int grid, int fmt) {
  return fmt == kFmtE2m1 ? launch_mode<MODE, kFmtE2m1>(L, tx, p, grid) : launch_mode<MODE, kFmtInt4>(L, tx, p, grid);
}

}  // namespace

bool gemm_w4a16_decode_applies(const GemmW4Args& a) {
  // grouped calls whose groups average at most 32 rows (decode batches)
  return a.offsets != nullptr && a.rows_total <= static_cast<int64_t>(NT) * a.E;
}

cudaError_t launch_gemm_w4a16_decode(const Launch& L, EncodeTiledFn encode, const GemmW4Args& a, CUresult* cu_err) {
  *cu_err = CUDA_SUCCESS;
  if (a.rows_total == 0) return cudaSuccess;
  CUtensorMap tx;
  CUresult r = make_tmap_x(encode, &tx, a.a_bf16, static_cast<uint64_t>(a.rows_total), static_cast<uint64_t>(a.K));
  if (r != CUDA_SUCCESS) {
    *cu_err = r;
    return cudaErrorUnknown;
  }
  W4DecodeParams p{};
  p.b_packed = a.b_packed;
  p.b_scales = a.b_scales;
  p.b_zeros = a.b_zeros;
  p.offsets = a.offsets;
  p.rows_total = static_cast<int>(a.rows_total);
  p.ksteps = static_cast<int>(a.K / BK);
  p.N = static_cast<int>(a.N);
  p.E = static_cast<int>(a.E);
  p.I = static_cast<int>(a.N / 2);
  p.n_pairs = a.mode == kModeGateUp ? static_cast<int>(a.N / 2 / BW) : static_cast<int>((a.N + 2 * BW - 1) / (2 * BW));
  p.out_bf16 = a.out_bf16;
  p.out_f32 = a.out_f32;
  p.h_bf16 = a.h_bf16;
  p.sorted_pair = a.sorted_pair;
  p.pair_weights = a.pair_weights;
  p.status = L.d_status;
  p.wait_limit_ns = L.wait_limit_ns ? L.wait_limit_ns : 2000000000ull;
  // upper bound on the tile count (group sizes live on the device): each expert adds at most one partial chunk
  const int64_t chunks_max = a.rows_total / NT + a.E;
  const int grid = static_cast<int>(std::min<int64_t>(L.sm_count, chunks_max * p.n_pairs));
  switch (a.mode) {
    case kModeLinear: return launch_fmt<kModeLinear>(L, tx, p, grid, a.fmt);
    case kModeGateUp: return launch_fmt<kModeGateUp>(L, tx, p, grid, a.fmt);
    case kModeDown: return launch_fmt<kModeDown>(L, tx, p, grid, a.fmt);
  }
  return cudaErrorInvalidValue;
}

}  // namespace qarl
