// Dense bf16 GEMM for sm_100a: the full-precision backward of the quantized linear layer
// (Sec. 3.1 item 2: low-bit forward, backward in full precision on the bf16 master weights,
// gradients passed through the quantizer by the straight-through estimator).
//
//   C[i, j] = sum over c ascending of A(i, c) * B(j, c),   fp32 accumulation in TMEM.
//
// Each operand is given as a row-major bf16 matrix in one of two orientations:
//   K-major   memory [rows = i or j][cols = c]   (the contraction index is contiguous)
//   MN-major  memory [rows = c][cols = i or j]   (the output index is contiguous)
// so that no transposed copy of dY, X or W is ever made:
//   dX[m, k] = sum_n dY[m, n] W[n, k]:  A = dY (K-major),  B = W  (MN-major, [c = n][j = k])
//   dW[n, k] = sum_m dY[m, n] X[m, k]:  A = dY (MN-major, [c = m][i = n]),  B = X (MN-major)
//
// Two grouped forms serve the expert GEMMs of the MoE layer, both on the forward's expert-sorted
// row layout (expert e owns rows offsets[e] .. offsets[e+1]-1), with no padding and no copies:
//   grouped rows         C[p, :] = A[p, :] . B_e  for the expert e that owns row p  (dX of an
//                        expert projection: A = dY sorted, K-major; B = W [E, N, K], MN-major)
//   grouped contraction  C_e = sum over the expert's rows p of A[p, :]^T B[p, :]  (dW of an
//                        expert projection: both operands MN-major, the contraction runs over a
//                        ragged row range).  The last 64-row step of an expert also holds rows of
//                        the next expert: the MMA warp overwrites those rows of the staged A tile
//                        with zeros (generic stores + proxy fence) before it issues the step, so
//                        they contribute nothing whatever B holds there.
//
// Tile 128 x 256 x 64.  TMA stages both operands with the 128-byte swizzle (a K-major tile is
// one box of R rows x 128 bytes; an MN-major tile is one box of 64 c-rows x 128 bytes per 64
// output indices); one thread issues 4 x tcgen05.mma kind::f16 (128 x 256 x 16) per stage with
// the matching operand-major bits; two 256-column TMEM accumulators let the epilogue of a tile
// overlap the main loop of the next.  Static persistent schedule, row tiles fastest.  One fixed
// order of accumulation: a result does not depend on the grid or on the other rows.
// Every wait is bounded (status word + CTA-wide abort flag), as in the other GEMMs.
#include <algorithm>
#include <atomic>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "sched.cuh"

namespace qarl {
namespace {

using namespace ptx;

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int kMaxStages = 4, kMaxAccBufs = 2;
constexpr int kEpiWarps = 4;   // warps 0-3 (TMEM quadrant = warp index)
constexpr int kTmaWarp = 4;
constexpr int kMmaWarp = 5;
constexpr int kThreads = 6 * 32;
constexpr uint32_t kAHalfBytes = BM * BK * 2;   // 16 KB: 128 output rows x 64 contraction elements
constexpr uint32_t kBBytes = BN * BK * 2;   // 32 KB
// A tile holds MT x 128 output rows.  The kernel is bound by the bytes it can keep in flight from
// L2/HBM (shared-memory capacity over load latency: throughput grew linearly with the ring depth),
// so MT = 2 -- both 128-row halves share one B tile, a third fewer bytes per flop -- is the default;
// it leaves one set of accumulators, i.e. an epilogue that is not overlapped, which only pays when
// the contraction is long enough (MT = 1 for the ragged contraction of the grouped dW).
template <int MT>
struct Cfg {
  static constexpr int kRows = MT * BM;
  static constexpr uint32_t kABytes = MT * kAHalfBytes;
  static constexpr uint32_t kStageBytes = kABytes + kBBytes;
  static constexpr int kStages = MT == 1 ? 4 : 3;
  static constexpr int kAccBufs = MT == 1 ? 2 : 1;
};
constexpr uint32_t kBlockBytes = 64 * BK * 2;  // one MN-major block: 64 output indices x 64 c-rows
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxExperts = 1024;
enum { kDense = 0, kGroupedRows = 1, kGroupedContraction = 2 };

struct Bf16Params {
  int Mo, No, Kc;           // grouped rows: Mo = total rows P;  grouped contraction: Kc unused (from offsets)
  const int32_t* offsets;   // [E + 1] (grouped forms)
  int E;
  int rows_total;           // grouped contraction: P
  int a3d, b3d;             // MN-major operand staged by one 3-D TMA box (64 columns x 64 rows x blocks)
  int col_fastest;          // dense: consecutive tiles walk the column tiles of a row tile (else the row tiles of a column tile)
  const int32_t* out_rows;  // grouped rows: output row of each sorted row (nullptr: the row itself)
  uint16_t* c_bf16;   // [Mo, No] or nullptr
  float* c_f32;       // [Mo, No] or nullptr
  int* status;
  unsigned long long wait_limit_ns;
};

struct __align__(8) SmemTail {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t tmem_full[kMaxAccBufs];
  uint64_t tmem_empty[kMaxAccBufs];
  uint64_t teardown;
  uint32_t tmem_addr;
  int abort_flag;
  int32_t off[kMaxExperts + 1];
  int32_t prefix[kMaxExperts + 1];
};
template <int MT>
constexpr size_t smem_bytes() { return 1024 + static_cast<size_t>(Cfg<MT>::kStages) * Cfg<MT>::kStageBytes + sizeof(SmemTail); }
static_assert(smem_bytes<1>() <= 227 * 1024 && smem_bytes<2>() <= 227 * 1024, "shared memory budget");

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, SmemTail* s, const Bf16Params& p) {
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
__device__ __forceinline__ bool warp_wait_or_abort(uint64_t* bar, uint32_t parity, SmemTail* s, const Bf16Params& p) {
  return __all_sync(0xFFFFFFFFu, wait_or_abort(bar, parity, s, p) ? 1 : 0) != 0;
}

__device__ __forceinline__ uint32_t bf16x2_bits(float lo, float hi) {
  const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&b);
}

template <bool A_MN, bool B_MN, int GROUP, int MT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                 const Bf16Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  using C = Cfg<MT>;
  constexpr int kStages = C::kStages, kAccBufs = C::kAccBufs, TM = C::kRows;
  constexpr uint32_t kABytes = C::kABytes, kStageBytes = C::kStageBytes;
  SmemTail* s = reinterpret_cast<SmemTail*>(smem + static_cast<size_t>(kStages) * kStageBytes);
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
    prefetch_tensormap(&tm_a);
    prefetch_tensormap(&tm_b);
  }
  if (warp == kMmaWarp) {
    tmem_alloc(&s->tmem_addr, kTmemCols);
    tmem_relinquish();
  }
  pdl_wait();
  const int n_tiles = (p.No + BN - 1) / BN;
  const int m_tiles = GROUP == kGroupedRows ? 1 : (p.Mo + TM - 1) / TM;  // grouped rows: tiles come from the offsets
  if (GROUP == kGroupedRows) {
    build_tile_list(s->off, s->prefix, p.offsets, p.Mo, p.E, TM, n_tiles);
  } else if (GROUP == kGroupedContraction) {
    for (int e = threadIdx.x; e <= p.E; e += kThreads) s->off[e] = min(max(p.offsets[e], 0), p.rows_total);
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = s->tmem_addr;
  const int total_tiles = GROUP == kGroupedRows ? s->prefix[p.E]
                        : GROUP == kGroupedContraction ? p.E * m_tiles * n_tiles : m_tiles * n_tiles;
  const int grid = gridDim.x;

  // Everything a role needs to know about tile T.  i0 / j0: first output row / column; a_c0 / b_c0:
  // first contraction coordinate of A / B; KS: 64-element contraction steps; last_valid: contraction
  // elements of the last step that belong to this tile (64 = all); row_end: end of the rows that
  // may be stored; c_off: element offset of this tile's output matrix.
  struct Tile {
    int i0, j0, a_c0, b_c0, KS, last_valid, row_end;
    int64_t c_off;
    int b_row0;  // K-major B: first row of the expert's block
  };
  auto tile_of = [&](int T, int& cur_e) {
    Tile t{};
    t.last_valid = BK;
    if (GROUP == kDense) {
      // CTAs that run at the same time take consecutive T.  Walking the column tiles of one row tile
      // together (col_fastest) lets a wave of CTAs read each block of A once and share it through L2;
      // walking the row tiles of one column tile together does the same for B.  The host picks the
      // order that re-reads the smaller operand.
      if (p.col_fastest) {
        t.i0 = (T / n_tiles) * TM;
        t.j0 = (T % n_tiles) * BN;
      } else {
        t.i0 = (T % m_tiles) * TM;
        t.j0 = (T / m_tiles) * BN;
      }
      t.KS = (p.Kc + BK - 1) / BK;  // a ragged last step reads zeros (TMA out-of-range fill)
      t.row_end = p.Mo;
    } else if (GROUP == kGroupedRows) {
      const TileCoord c = decode_tile(s->off, s->prefix, TM, T, cur_e);
      t.i0 = c.m0;
      t.j0 = c.n_tile * BN;
      t.KS = p.Kc / BK;             // Kc is a multiple of 64 here: a step never runs into the next expert's weights
      t.a_c0 = 0;
      t.b_c0 = c.e * p.Kc;          // MN-major B: the expert's [Kc, No] block starts at row e Kc
      t.b_row0 = c.e * p.No;        // K-major B: the expert's [No, Kc] block starts at row e No
      t.row_end = c.m_end;
    } else {
      const int per_e = m_tiles * n_tiles;
      const int e = T / per_e, r = T % per_e;
      t.i0 = (r % m_tiles) * TM;
      t.j0 = (r / m_tiles) * BN;
      const int rows = s->off[e + 1] - s->off[e];
      t.KS = (rows + BK - 1) / BK;
      t.last_valid = rows - (t.KS - 1) * BK;
      t.a_c0 = t.b_c0 = s->off[e];
      t.row_end = p.Mo;
      t.c_off = static_cast<int64_t>(e) * p.Mo * p.No;
    }
    return t;
  };

  if (warp == kTmaWarp) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t armed = 0, armed_parity = 0;
      bool ok = true;
      int cur_e = 0;
      for (int T = blockIdx.x; ok && T < total_tiles; T += grid) {
        const Tile t = tile_of(T, cur_e);
        const int i0 = t.i0, j0 = t.j0;
        for (int ks = 0; ks < t.KS; ++ks) {
          if (!wait_or_abort(&s->empty[stage], phase ^ 1, s, p)) { ok = false; break; }
          uint8_t* a_dst = smem + static_cast<size_t>(stage) * kStageBytes;
          uint8_t* b_dst = a_dst + kABytes;
          mbar_arrive_expect_tx(&s->full[stage], kStageBytes);
          if (A_MN && p.a3d) {
            tma_load_3d(a_dst, &tm_a, &s->full[stage], 0, t.a_c0 + ks * BK, i0 / 64);
          } else if (A_MN) {
#pragma unroll
            for (int b = 0; b < TM / 64; ++b)
              tma_load_2d(a_dst + b * kBlockBytes, &tm_a, &s->full[stage], i0 + 64 * b, t.a_c0 + ks * BK);
          } else {  // one box of TM rows x 128 bytes
            tma_load_2d(a_dst, &tm_a, &s->full[stage], t.a_c0 + ks * BK, i0);
          }
          if (B_MN && p.b3d) {
            tma_load_3d(b_dst, &tm_b, &s->full[stage], 0, t.b_c0 + ks * BK, j0 / 64);
          } else if (B_MN) {
#pragma unroll
            for (int b = 0; b < BN / 64; ++b)
              tma_load_2d(b_dst + b * kBlockBytes, &tm_b, &s->full[stage], j0 + 64 * b, t.b_c0 + ks * BK);
          } else {
            tma_load_2d(b_dst, &tm_b, &s->full[stage], ks * BK, t.b_row0 + j0);
          }
          armed |= 1u << stage;
          armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        for (int i = 0; i < kStages; ++i)
          if (armed & (1u << i)) mbar_wait_bounded(&s->full[i], (armed_parity >> i) & 1u, 20000000ull);
      }
    }
  } else if (warp == kMmaWarp) {
    // The whole warp follows the pipeline (so that it can zero the overhang rows of a ragged
    // contraction step together); lane 0 issues the MMAs and commits.
    constexpr uint32_t idesc = umma_idesc_bf16_f32_major(BM, BN, A_MN, B_MN);
    int stage = 0, acc = 0;
    uint32_t phase = 0, acc_phase = 0;
    bool ok = true;
    int cur_e = 0;
    for (int T = blockIdx.x; ok && T < total_tiles; T += grid) {
      const Tile t = tile_of(T, cur_e);
      if (t.KS == 0) continue;  // an expert without rows: the epilogue writes zeros, no accumulator is used
      if (!warp_wait_or_abort(&s->tmem_empty[acc], acc_phase ^ 1, s, p)) { ok = false; break; }
      const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * MT) * BN;
      for (int ks = 0; ks < t.KS; ++ks) {
        if (!warp_wait_or_abort(&s->full[stage], phase, s, p)) { ok = false; break; }
        uint8_t* a_tile = smem + static_cast<size_t>(stage) * kStageBytes;
        if (GROUP == kGroupedContraction && ks == t.KS - 1 && t.last_valid < BK) {
          // rows last_valid .. 63 of both 64-column blocks of A belong to the next expert: make them zero
          const int nrows = BK - t.last_valid;
          for (int idx = lane; idx < (TM / 64) * nrows * 8; idx += 32) {
            const int blk = idx / (nrows * 8), rem = idx % (nrows * 8);
            *reinterpret_cast<uint4*>(a_tile + blk * kBlockBytes + (t.last_valid + rem / 8) * 128 + (rem % 8) * 16) =
                make_uint4(0, 0, 0, 0);
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        __syncwarp();
        if (lane == 0) {
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(a_tile);
          const uint32_t b_addr = a_addr + kABytes;
          const uint64_t a_desc = A_MN ? umma_desc_mn_sw128(a_addr, kBlockBytes) : umma_desc_k_sw128(a_addr);
          const uint64_t b_desc = B_MN ? umma_desc_mn_sw128(b_addr, kBlockBytes) : umma_desc_k_sw128(b_addr);
          // 16 contraction elements further on: 32 bytes inside a K-major row, 16 rows of 128 bytes
          // in an MN-major block (start-address field counts 16-byte units)
          constexpr uint32_t a_step = A_MN ? (16 * 128) >> 4 : 32 >> 4;
          constexpr uint32_t b_step = B_MN ? (16 * 128) >> 4 : 32 >> 4;
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)  // the 128-row halves of A share the B tile
#pragma unroll
            for (int k4 = 0; k4 < BK / 16; ++k4)
              umma_bf16(d_tmem + mt * BN, a_desc + mt * (kAHalfBytes >> 4) + a_step * k4, b_desc + b_step * k4, idesc,
                        (ks > 0 || k4 > 0) ? 1u : 0u);
          umma_commit(&s->empty[stage]);
          if (ks == t.KS - 1) umma_commit(&s->tmem_full[acc]);
        }
        __syncwarp();
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
      if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1; }
    }
    // Nothing of this CTA's tensor work may be in flight when its TMEM and shared memory go
    // away: after an abort some MMAs may still be executing, so wait (bounded) for them.
    if (!ok && lane == 0) {
      umma_commit(&s->teardown);
      mbar_wait_bounded(&s->teardown, 0, 20000000ull);
    }
  } else if (warp < kEpiWarps) {
    const int r = warp * 32 + lane;
    const uint32_t lane_addr = static_cast<uint32_t>(warp * 32) << 16;
    int acc = 0;
    uint32_t acc_phase = 0;
    int cur_e = 0;
    for (int T = blockIdx.x; T < total_tiles; T += grid) {
      const Tile t = tile_of(T, cur_e);
      const int j0 = t.j0;
      const bool have_acc = t.KS > 0;
      if (have_acc) {
        if (!warp_wait_or_abort(&s->tmem_full[acc], acc_phase, s, p)) break;
        tc_fence_after_sync();
      }
#pragma unroll 1
      for (int mt = 0; mt < MT; ++mt) {
      const int i0 = t.i0 + mt * BM;
      const int row = i0 + r;
      const bool valid = row < t.row_end;
      const bool warp_live = i0 + warp * 32 < t.row_end;
      const uint32_t t0 = tmem_base + lane_addr + static_cast<uint32_t>((acc * MT + mt) * BN);
      if (warp_live) {
#pragma unroll 1
        for (int ch = 0; ch < BN / 16; ++ch) {
          const int col = j0 + 16 * ch;
          if (col >= p.No) break;
          uint32_t v[16];
          if (have_acc) {
            tmem_ld_x16(t0 + 16 * ch, v);
            tmem_ld_wait();
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = 0u;
          }
          if (valid) {
            const bool whole = col + 16 <= p.No;  // No is a multiple of 8: a ragged last chunk holds 8 columns
            int64_t orow = row;
            if (GROUP == kGroupedRows && p.out_rows) orow = min(max(__ldg(p.out_rows + row), 0), p.Mo - 1);
            const int64_t at = t.c_off + orow * p.No + col;
            if (p.c_f32) {
              float4* fd = reinterpret_cast<float4*>(p.c_f32 + at);
#pragma unroll
              for (int j = 0; j < 4; ++j)
                if (j < 2 || whole)
                  fd[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                      __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
            }
            if (p.c_bf16) {
              uint32_t ob[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) ob[j] = bf16x2_bits(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
              uint4* od = reinterpret_cast<uint4*>(p.c_bf16 + at);
              od[0] = make_uint4(ob[0], ob[1], ob[2], ob[3]);
              if (whole) od[1] = make_uint4(ob[4], ob[5], ob[6], ob[7]);
            }
          }
        }
      }
      }  // mt
      if (have_acc) {
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s->tmem_empty[acc]);
        if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1; }
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Tensor map of a row-major bf16 matrix [rows, cols] with a box of box_cols x box_rows elements.
CUresult make_tmap(EncodeTiledFn encode, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                   uint32_t box_cols, uint32_t box_rows) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// An MN-major matrix [rows, cols] (cols % 64 == 0) seen as 64-column blocks: dims {64, rows, cols / 64};
// one box of 64 x 64 x nblocks lands as nblocks consecutive 8 KB blocks, the layout the descriptor expects.
// The issuing thread pays per TMA instruction, so one box per operand instead of one per block matters.
CUresult make_tmap_mn3d(EncodeTiledFn encode, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                        uint32_t nblocks) {
  const cuuint64_t dims[3] = {64, rows, cols / 64};
  const cuuint64_t strides[2] = {cols * 2, 128};
  const cuuint32_t box[3] = {64, BK, nblocks};
  const cuuint32_t estr[3] = {1, 1, 1};
  return encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

template <bool A_MN, bool B_MN, int GROUP, int MT>
cudaError_t launch_variant(const Launch& L, const CUtensorMap& ta, const CUtensorMap& tb, const Bf16Params& p,
                           int64_t tiles) {
  // sticky per function and device; atomic: contexts on several host threads may launch at once (both
  // would set the same value)
  static std::atomic<bool> attr_set_dev[64];
  std::atomic<bool>& attr_set = attr_set_dev[L.device & 63];
  if (!attr_set.load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_bf16_kernel<A_MN, B_MN, GROUP, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem_bytes<MT>()));
    if (e != cudaSuccess) return e;
    attr_set.store(true, std::memory_order_release);
  }
  // full rounds only: with W = ceil(tiles / SMs) rounds, ceil(tiles / W) CTAs finish in W rounds
  // (for grouped rows `tiles` is an upper bound: the surplus CTAs find no tile and retire)
  const int64_t rounds = std::max<int64_t>(1, (tiles + L.sm_count - 1) / L.sm_count);
  const int grid = static_cast<int>(std::max<int64_t>(1, (tiles + rounds - 1) / rounds));
  ++*L.launches;
  return launch_pdl(gemm_bf16_kernel<A_MN, B_MN, GROUP, MT>, static_cast<unsigned>(grid), kThreads, smem_bytes<MT>(), L.stream, ta, tb, p);
}

}  // namespace

cudaError_t launch_gemm_bf16(const Launch& L, EncodeTiledFn encode, const GemmBf16Args& a, CUresult* cu_err) {
  *cu_err = CUDA_SUCCESS;
  if (a.Mo == 0 || a.No == 0) return cudaSuccess;
  const bool grouped_rows = a.group == 1, grouped_k = a.group == 2;
  // 256-row tiles pay (measured: 13 % less time per unit of work) when the tile count still fills the
  // SMs' rounds; the grouped forms keep 128-row tiles (ragged groups waste more of a 256-row tile and
  // the single accumulator set exposes the epilogue of short tiles).
  int MT = 1;
  if (a.group == 0 && a.Mo > BM) {
    const int64_t n_t = (a.No + BN - 1) / BN;
    const int64_t t1 = (a.Mo + BM - 1) / BM * n_t, t2 = (a.Mo + 2 * BM - 1) / (2 * BM) * n_t;
    const double cost1 = static_cast<double>((t1 + L.sm_count - 1) / L.sm_count);
    const double cost2 = static_cast<double>((t2 + L.sm_count - 1) / L.sm_count) * 2.0 * 0.87;
    if (cost2 < cost1) MT = 2;
  }
  const int TM = MT * BM;
  // rows of the tensors as TMA sees them
  const int64_t a_rows = a.a_mn_major ? (grouped_k ? a.rows_total : a.Kc) : a.Mo;
  const int64_t b_rows = a.b_mn_major ? (grouped_k ? a.rows_total : (grouped_rows ? a.E * a.Kc : a.Kc))
                                      : (grouped_rows ? a.E * a.No : a.No);
  CUtensorMap ta, tb;
  const bool a3d = a.a_mn_major && a.Mo % 64 == 0, b3d = a.b_mn_major && a.No % 64 == 0;
  CUresult r = a3d ? make_tmap_mn3d(encode, &ta, a.a, a_rows, a.Mo, TM / 64)
             : a.a_mn_major ? make_tmap(encode, &ta, a.a, a_rows, a.Mo, 64, BK) : make_tmap(encode, &ta, a.a, a_rows, a.Kc, BK, TM);
  if (r == CUDA_SUCCESS)
    r = b3d ? make_tmap_mn3d(encode, &tb, a.b, b_rows, a.No, BN / 64)
      : a.b_mn_major ? make_tmap(encode, &tb, a.b, b_rows, a.No, 64, BK) : make_tmap(encode, &tb, a.b, b_rows, a.Kc, BK, BN);
  if (r != CUDA_SUCCESS) {
    *cu_err = r;
    return cudaErrorUnknown;
  }
  Bf16Params p{};
  p.Mo = static_cast<int>(a.Mo);
  p.No = static_cast<int>(a.No);
  p.Kc = static_cast<int>(a.Kc);
  p.offsets = a.offsets;
  p.E = static_cast<int>(a.E);
  p.rows_total = static_cast<int>(a.rows_total);
  p.out_rows = a.out_rows;
  p.a3d = a3d;
  p.b3d = b3d;
  p.col_fastest = a.group == 0 && a.Mo >= a.No;  // A (Mo x Kc) is the larger operand: re-read B, not A
  p.c_bf16 = a.c_bf16;
  p.c_f32 = a.c_f32;
  p.status = L.d_status;
  p.wait_limit_ns = 2000000000ull;
  const int64_t n_tiles = (a.No + BN - 1) / BN;
  if (grouped_rows) {  // A K-major; each expert adds at most one partial row tile
    const int64_t tiles = (a.Mo / TM + a.E) * n_tiles;
    return a.b_mn_major ? launch_variant<false, true, kGroupedRows, 1>(L, ta, tb, p, tiles)
                        : launch_variant<false, false, kGroupedRows, 1>(L, ta, tb, p, tiles);
  }
  const int64_t m_tiles = (a.Mo + TM - 1) / TM;
  if (grouped_k) return launch_variant<true, true, kGroupedContraction, 1>(L, ta, tb, p, a.E * m_tiles * n_tiles);
  const int64_t tiles = m_tiles * n_tiles;
  if (MT == 2) {
    if (a.a_mn_major)
      return a.b_mn_major ? launch_variant<true, true, kDense, 2>(L, ta, tb, p, tiles) : launch_variant<true, false, kDense, 2>(L, ta, tb, p, tiles);
    return a.b_mn_major ? launch_variant<false, true, kDense, 2>(L, ta, tb, p, tiles) : launch_variant<false, false, kDense, 2>(L, ta, tb, p, tiles);
  }
  if (a.a_mn_major)
    return a.b_mn_major ? launch_variant<true, true, kDense, 1>(L, ta, tb, p, tiles) : launch_variant<true, false, kDense, 1>(L, ta, tb, p, tiles);
  return a.b_mn_major ? launch_variant<false, true, kDense, 1>(L, ta, tb, p, tiles) : launch_variant<false, false, kDense, 1>(L, ta, tb, p, tiles);
}

}  // namespace qarl
