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
// Structure of a CTA (576 threads, one CTA per SM, persistent over a static tile list):
//   warp 16   TMA producer: per K-block one stage = A box 128x128 B + two B boxes 128x128 B
//             (SWIZZLE_128B) into a 4-deep shared-memory ring;
//   warp 17   MMA issuer: 4 x tcgen05.mma kind::f8f6f4 per K-block into one of two 256-column
//             TMEM accumulators (overwrite on the first), then tcgen05.commit to free the
//             smem stage and to publish the accumulator;
//   warps 0-15 promotion + epilogue: warp w reads TMEM lanes 32*(w%4).. (its hardware
//             quadrant) and two 32-column slices, one in each 128-column half of the tile,
//             multiplies the block partial by the combined scale and adds it to fp32
//             registers; MMA of block kb+1 overlaps promotion of block kb.
// The two 128-column halves of a tile are rows [n_lo, n_lo+128) and [n_hi, n_hi+128) of the
// weight: adjacent for linear/down, gate rows and the matching up rows for gate_up so that
// SwiGLU and the 1x128 re-quantization of h happen in registers.
//
// Every wait on an mbarrier is bounded; on expiry the thread records
// QARL_ERR_DEVICE_TIMEOUT, raises a CTA-wide abort flag that all other waits poll, and the
// CTA drains and frees its TMEM, so a broken pipeline returns an error instead of hanging.
#include <algorithm>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace qarl {
namespace {

using namespace ptx;

constexpr int BM = 128;           // rows per tile (UMMA M)
constexpr int BNH = 128;          // columns per half tile
constexpr int BN = 2 * BNH;       // UMMA N
constexpr int BK = 128;           // one K-block = one 128-byte swizzle span of e4m3
constexpr int kStages = 4;
constexpr int kAccStages = 2;
constexpr int kEpiWarps = 16;
constexpr int kTmaWarp = 16;
constexpr int kMmaWarp = 17;
constexpr int kThreads = 18 * 32;
constexpr uint32_t kABytes = BM * BK;
constexpr uint32_t kBBytes = BN * BK;
constexpr uint32_t kStageBytes = kABytes + kBBytes;  // 48 KB
constexpr uint32_t kTmemCols = 512;
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
  uint16_t* out_bf16;
  float* out_f32;
  uint8_t* h_codes;
  float* h_scales;
  uint16_t* h_bf16;
  const int32_t* sorted_pair;
  const float* pair_weights;
  int* status;
  unsigned long long wait_limit_ns;
};

struct __align__(8) SmemTail {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t tmem_full[kAccStages];
  uint64_t tmem_empty[kAccStages];
  uint64_t amax_bar[2];
  uint32_t tmem_addr;
  int abort_flag;
  int32_t off[kMaxExperts + 1];
  int32_t prefix[kMaxExperts + 1];
  float amax[2][4][BM];
};

constexpr size_t kSmemBytes = 1024 + static_cast<size_t>(kStages) * kStageBytes + sizeof(SmemTail);

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

__device__ __forceinline__ float silu_mul(float g, float u) { return (g / (1.0f + __expf(-g))) * u; }

template <int MODE>
__global__ void __launch_bounds__(kThreads, 1)
gemm_blockscaled_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                        const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  SmemTail* s = reinterpret_cast<SmemTail*>(smem + static_cast<size_t>(kStages) * kStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- set-up: barriers, TMEM, tile list ------------------------------------------------
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&s->full[i], 1);
      mbar_init(&s->empty[i], 1);
    }
    for (int i = 0; i < kAccStages; ++i) {
      mbar_init(&s->tmem_full[i], 1);
      mbar_init(&s->tmem_empty[i], kEpiWarps);
    }
    mbar_init(&s->amax_bar[0], kEpiWarps);
    mbar_init(&s->amax_bar[1], kEpiWarps);
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
  for (int e = threadIdx.x; e <= p.E; e += kThreads)
    s->off[e] = p.offsets ? p.offsets[e] : (e == 0 ? 0 : p.rows_total);
  __syncthreads();
  if (warp == 0) {  // exclusive scan of tiles per expert
    int carry = 0;
    for (int base = 0; base < p.E; base += 32) {
      const int e = base + lane;
      int v = 0;
      if (e < p.E) v = ((s->off[e + 1] - s->off[e] + BM - 1) / BM) * p.n_tiles;
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
  const int KB = p.kblocks;
  const int NB = p.N / BNH;  // weight scale block-rows per expert

  if (warp == kTmaWarp) {
    // =============================== TMA producer =====================================
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t armed = 0, armed_parity = 0;  // per-stage: has a load in flight / its parity
      int cur_e = 0;
      bool ok = true;
      for (int T = blockIdx.x; ok && T < total_tiles; T += gridDim.x) {
        const TileCoord c = decode_tile(s, T, cur_e);
        int row_lo, row_hi;
        if (MODE == kModeGateUp) {
          row_lo = c.e * p.N + c.n_tile * BNH;
          row_hi = row_lo + p.I;
        } else {
          row_lo = c.e * p.N + c.n_tile * BN;
          row_hi = row_lo + BNH;
        }
        for (int kb = 0; kb < KB; ++kb) {
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
  } else if (warp == kMmaWarp) {
    // =============================== MMA issuer =======================================
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_e4m3_f32(BM, BN);
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int T = blockIdx.x; ok && T < total_tiles; T += gridDim.x) {
        for (int kb = 0; kb < KB; ++kb) {
          if (!wait_or_abort(&s->tmem_empty[acc], acc_phase ^ 1, s, p)) { ok = false; break; }
          if (!wait_or_abort(&s->full[stage], phase, s, p)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(smem + static_cast<size_t>(stage) * kStageBytes);
          const uint64_t a_desc = umma_desc_k_sw128(a_addr);
          const uint64_t b_desc = umma_desc_k_sw128(a_addr + kABytes);
          const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc) * BN;
#pragma unroll
          for (int k4 = 0; k4 < BK / 32; ++k4)  // +32 bytes of K = +2 in the 16-byte address field
            umma_f8(d_tmem, a_desc + 2 * k4, b_desc + 2 * k4, idesc, k4 > 0 ? 1u : 0u);
          umma_commit(&s->empty[stage]);
          umma_commit(&s->tmem_full[acc]);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
          if (++acc == kAccStages) { acc = 0; acc_phase ^= 1; }
        }
      }
    }
  } else {
    // =============================== promotion + epilogue =============================
    const int q = warp & 3;          // TMEM lane quadrant this warp may read
    const int cg = warp >> 2;        // 32-column slice within each half tile
    const int r = q * 32 + lane;     // row within the tile
    const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
    int acc = 0;
    uint32_t acc_phase = 0;
    int cur_e = 0;
    uint32_t tile_iter = 0;      // tiles this CTA has finished (selects the amax exchange buffer)
    bool ok = true;
    for (int T = blockIdx.x; ok && T < total_tiles; T += gridDim.x) {
      const TileCoord c = decode_tile(s, T, cur_e);
      const int row = c.m0 + r;
      const bool valid = row < c.m_end;
      const int row_c = min(row, p.rows_total - 1);
      int nb_lo, nb_hi;
      if (MODE == kModeGateUp) {
        nb_lo = c.n_tile;
        nb_hi = c.n_tile + p.I / BNH;
      } else {
        nb_lo = 2 * c.n_tile;
        nb_hi = min(2 * c.n_tile + 1, NB - 1);
      }
      const float* sx_ptr = p.a_scales + static_cast<int64_t>(row_c) * KB;
      const float* sw_lo_ptr = p.b_scales + (static_cast<int64_t>(c.e) * NB + nb_lo) * KB;
      const float* sw_hi_ptr = p.b_scales + (static_cast<int64_t>(c.e) * NB + nb_hi) * KB;

      float acc_lo[32], acc_hi[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) acc_lo[j] = acc_hi[j] = 0.0f;

      float sx_next = __ldg(sx_ptr), swl_next = __ldg(sw_lo_ptr), swh_next = __ldg(sw_hi_ptr);
      for (int kb = 0; kb < KB; ++kb) {
        const float sc_lo = __fmul_rn(sx_next, swl_next);
        const float sc_hi = __fmul_rn(sx_next, swh_next);
        if (kb + 1 < KB) {
          sx_next = __ldg(sx_ptr + kb + 1);
          swl_next = __ldg(sw_lo_ptr + kb + 1);
          swh_next = __ldg(sw_hi_ptr + kb + 1);
        }
        if (!wait_or_abort(&s->tmem_full[acc], acc_phase, s, p)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t t_lo = tmem_base + lane_addr + static_cast<uint32_t>(acc * BN + cg * 32);
        const uint32_t t_hi = t_lo + BNH;
        uint32_t v0[16], v1[16];
        tmem_ld_x16(t_lo, v0);
        tmem_ld_wait();
        tmem_ld_x16(t_lo + 16, v1);
#pragma unroll
        for (int j = 0; j < 16; ++j) acc_lo[j] = __fmaf_rn(sc_lo, __uint_as_float(v0[j]), acc_lo[j]);
        tmem_ld_wait();
        tmem_ld_x16(t_hi, v0);
#pragma unroll
        for (int j = 0; j < 16; ++j) acc_lo[16 + j] = __fmaf_rn(sc_lo, __uint_as_float(v1[j]), acc_lo[16 + j]);
        tmem_ld_wait();
        tmem_ld_x16(t_hi + 16, v1);
#pragma unroll
        for (int j = 0; j < 16; ++j) acc_hi[j] = __fmaf_rn(sc_hi, __uint_as_float(v0[j]), acc_hi[j]);
        tmem_ld_wait();
        // all of this warp's reads of the accumulator are done: hand it back to the MMA warp
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s->tmem_empty[acc]);
#pragma unroll
        for (int j = 0; j < 16; ++j) acc_hi[16 + j] = __fmaf_rn(sc_hi, __uint_as_float(v1[j]), acc_hi[16 + j]);
        if (++acc == kAccStages) { acc = 0; acc_phase ^= 1; }
      }
      if (!ok) break;

      // ---- tile epilogue ------------------------------------------------------------------
      if (MODE == kModeLinear || MODE == kModeDown) {
        const int col_lo = c.n_tile * BN + cg * 32;
        const int col_hi = col_lo + BNH;
        const bool hi_valid = col_hi < p.N;
        if (valid) {
          int64_t out_row = row;
          float w = 1.0f;
          if (MODE == kModeDown) {
            const int pair = __ldg(p.sorted_pair + row);
            out_row = pair;
            w = __ldg(p.pair_weights + pair);
          }
          if (p.out_f32) {
            float4* d_lo = reinterpret_cast<float4*>(p.out_f32 + static_cast<int64_t>(row) * p.N + col_lo);
            float4* d_hi = reinterpret_cast<float4*>(p.out_f32 + static_cast<int64_t>(row) * p.N + col_hi);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              d_lo[j] = make_float4(acc_lo[4 * j], acc_lo[4 * j + 1], acc_lo[4 * j + 2], acc_lo[4 * j + 3]);
              if (hi_valid)
                d_hi[j] = make_float4(acc_hi[4 * j], acc_hi[4 * j + 1], acc_hi[4 * j + 2], acc_hi[4 * j + 3]);
            }
          }
          uint4* o_lo = reinterpret_cast<uint4*>(p.out_bf16 + out_row * p.N + col_lo);
          uint4* o_hi = reinterpret_cast<uint4*>(p.out_bf16 + out_row * p.N + col_hi);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint4 a, b;
            if (MODE == kModeDown) {
              a.x = pack_bf16x2(__fmul_rn(w, acc_lo[8 * j + 0]), __fmul_rn(w, acc_lo[8 * j + 1]));
              a.y = pack_bf16x2(__fmul_rn(w, acc_lo[8 * j + 2]), __fmul_rn(w, acc_lo[8 * j + 3]));
              a.z = pack_bf16x2(__fmul_rn(w, acc_lo[8 * j + 4]), __fmul_rn(w, acc_lo[8 * j + 5]));
              a.w = pack_bf16x2(__fmul_rn(w, acc_lo[8 * j + 6]), __fmul_rn(w, acc_lo[8 * j + 7]));
              b.x = pack_bf16x2(__fmul_rn(w, acc_hi[8 * j + 0]), __fmul_rn(w, acc_hi[8 * j + 1]));
              b.y = pack_bf16x2(__fmul_rn(w, acc_hi[8 * j + 2]), __fmul_rn(w, acc_hi[8 * j + 3]));
              b.z = pack_bf16x2(__fmul_rn(w, acc_hi[8 * j + 4]), __fmul_rn(w, acc_hi[8 * j + 5]));
              b.w = pack_bf16x2(__fmul_rn(w, acc_hi[8 * j + 6]), __fmul_rn(w, acc_hi[8 * j + 7]));
            } else {
              a.x = pack_bf16x2(acc_lo[8 * j + 0], acc_lo[8 * j + 1]);
              a.y = pack_bf16x2(acc_lo[8 * j + 2], acc_lo[8 * j + 3]);
              a.z = pack_bf16x2(acc_lo[8 * j + 4], acc_lo[8 * j + 5]);
              a.w = pack_bf16x2(acc_lo[8 * j + 6], acc_lo[8 * j + 7]);
              b.x = pack_bf16x2(acc_hi[8 * j + 0], acc_hi[8 * j + 1]);
              b.y = pack_bf16x2(acc_hi[8 * j + 2], acc_hi[8 * j + 3]);
              b.z = pack_bf16x2(acc_hi[8 * j + 4], acc_hi[8 * j + 5]);
              b.w = pack_bf16x2(acc_hi[8 * j + 6], acc_hi[8 * j + 7]);
            }
            o_lo[j] = a;
            if (hi_valid) o_hi[j] = b;
          }
        }
      } else {
        // gate_up: lo half = gate columns, hi half = the matching up columns.
        const int col = c.n_tile * BNH + cg * 32;  // column of h (and of gate) in [0, I)
        uint32_t hb[16];                           // 32 bf16 values of h, packed in pairs
        float amax = 0.0f;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const uint32_t g2 = pack_bf16x2(acc_lo[2 * j], acc_lo[2 * j + 1]);
          const uint32_t u2 = pack_bf16x2(acc_hi[2 * j], acc_hi[2 * j + 1]);
          const float h0 = silu_mul(bf16_bits_to_f32(g2 & 0xFFFFu), bf16_bits_to_f32(u2 & 0xFFFFu));
          const float h1 = silu_mul(bf16_bits_to_f32(g2 >> 16), bf16_bits_to_f32(u2 >> 16));
          hb[j] = pack_bf16x2(h0, h1);
          amax = fmaxf(amax, fmaxf(fabsf(bf16_bits_to_f32(hb[j] & 0xFFFFu)), fabsf(bf16_bits_to_f32(hb[j] >> 16))));
          if (p.out_bf16 && valid) {  // debug dump of the bf16 gate_up row
            p.out_bf16[static_cast<int64_t>(row) * p.N + col + 2 * j] = static_cast<uint16_t>(g2 & 0xFFFFu);
            p.out_bf16[static_cast<int64_t>(row) * p.N + col + 2 * j + 1] = static_cast<uint16_t>(g2 >> 16);
            p.out_bf16[static_cast<int64_t>(row) * p.N + p.I + col + 2 * j] = static_cast<uint16_t>(u2 & 0xFFFFu);
            p.out_bf16[static_cast<int64_t>(row) * p.N + p.I + col + 2 * j + 1] = static_cast<uint16_t>(u2 >> 16);
          }
        }
        // the 128-wide quantization group of this row spans the 4 column slices (4 warps)
        // (double-buffered by tile so that a fast warp cannot overwrite values still being read)
        const uint32_t xb = tile_iter & 1u;
        s->amax[xb][cg][r] = amax;
        __syncwarp();
        if (lane == 0) mbar_arrive(&s->amax_bar[xb]);
        if (!wait_or_abort(&s->amax_bar[xb], (tile_iter >> 1) & 1u, s, p)) break;
        amax = fmaxf(fmaxf(s->amax[xb][0][r], s->amax[xb][1][r]), fmaxf(s->amax[xb][2][r], s->amax[xb][3][r]));
        float inv;
        const float sc = block_scale(amax, &inv);
        if (valid) {
          uint32_t cw[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float f0 = __fmul_rn(bf16_bits_to_f32(hb[2 * j] & 0xFFFFu), inv);
            const float f1 = __fmul_rn(bf16_bits_to_f32(hb[2 * j] >> 16), inv);
            const float f2 = __fmul_rn(bf16_bits_to_f32(hb[2 * j + 1] & 0xFFFFu), inv);
            const float f3 = __fmul_rn(bf16_bits_to_f32(hb[2 * j + 1] >> 16), inv);
            cw[j] = cvt_e4m3x4(f0, f1, f2, f3);
          }
          uint4* dst = reinterpret_cast<uint4*>(p.h_codes + static_cast<int64_t>(row) * p.I + col);
          dst[0] = make_uint4(cw[0], cw[1], cw[2], cw[3]);
          dst[1] = make_uint4(cw[4], cw[5], cw[6], cw[7]);
          if (cg == 0) p.h_scales[static_cast<int64_t>(row) * (p.I / BNH) + c.n_tile] = sc;
          if (p.h_bf16) {
            uint4* hd = reinterpret_cast<uint4*>(p.h_bf16 + static_cast<int64_t>(row) * p.I + col);
#pragma unroll
            for (int j = 0; j < 4; ++j) hd[j] = make_uint4(hb[4 * j], hb[4 * j + 1], hb[4 * j + 2], hb[4 * j + 3]);
          }
        }
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
  static bool attr_set_dev[64] = {};  // the attribute is sticky per function and device
  bool& attr_set = attr_set_dev[L.device & 63];
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(gemm_blockscaled_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kSmemBytes));
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  gemm_blockscaled_kernel<MODE><<<grid, kThreads, kSmemBytes, L.stream>>>(ta, tb, p);
  ++*L.launches;
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_gemm(const Launch& L, EncodeTiledFn encode, const GemmArgs& a, CUresult* cu_err) {
  *cu_err = CUDA_SUCCESS;
  if (a.rows_total == 0) return cudaSuccess;
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
  p.wait_limit_ns = 2000000000ull;
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
