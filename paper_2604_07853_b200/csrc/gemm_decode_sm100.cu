// Block-scaled FP8 grouped GEMM for decode-sized row groups (a few tokens per expert): the same
// arithmetic as gemm_sm100.cu with the operands of the MMA swapped.
//
// With ~16 rows per expert a 128-row token tile is almost empty, and the kernel is bound by the
// per-K-block round trip between the MMA and the promotion warps, not by the weight stream it is
// supposed to be bound by (Appendix D.1: MoE decode is memory-bound).  Here the 128 WEIGHT rows of
// a scale block are the M side of tcgen05.mma and at most 32 TOKEN rows are its N side:
//   D[w, t] = sum_k W_q[w, k] X_q[t, k]      (kind::f8f6f4, M = 128, N = 32, K = 32, four per K-block)
// The products are exact and the instruction adds them in the same order whichever operand carries
// which matrix (verified bit for bit on the device over 10^8 random dot products, N = 16 ... 128),
// so p_kb[t, w] has the bits the wide kernel computes, and the promotion
//   acc[t, w] = fmaf( fl(s_x[t,kb] * s_w[w/128,kb]), p_kb[t, w], acc[t, w] ),  kb ascending from 0.0f
// is the same chain: a token's output row is bitwise the same in both kernels (the row-invariance
// tests and the 48-layer alignment stack compare them).  An MMA of N = 32 costs an eighth of the
// wide one, an accumulator is 64 TMEM columns (gate + up, or two adjacent weight blocks), so eight
// accumulators are in flight and the weight stream (5 stages of 36 KB per SM) is what remains.
//
// A tile = (expert e, pair of weight blocks j, chunk of <= 32 rows of the expert's group):
//   gate_up: blocks j (gate rows) and j + I/128 (the matching up rows); down/linear: blocks 2j, 2j+1.
// CTA = 192 threads: warps 0-3 promotion + epilogue (thread = weight row, 2 x 32 accumulators),
// warp 4 TMA producer, warp 5 MMA issuer.  The epilogue transposes through shared memory so that
// global stores are whole rows: gate_up applies SwiGLU in registers (gate and up of an element sit
// in the same thread), then a warp per token row does the 1x128 amax / scale / e4m3 codes; down
// multiplies by the pair's combine weight and writes bf16 contribution rows.
// Every barrier wait is bounded as in the wide kernel; an expired wait aborts the CTA cleanly.
#include <algorithm>
#include <atomic>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "sched.cuh"

namespace qarl {
namespace {

using namespace ptx;

constexpr int BW = 128;           // weight rows per MMA (UMMA M) = one scale block
constexpr int NT = 32;            // token rows per tile (UMMA N)
constexpr int BK = 128;
constexpr int kStages = 5;         // 36 KB each: 180 KB of loads in flight per SM (2, 3, 5 stages: 99, 92, 87 us at decode)
constexpr int kAccBufs = 8;       // TMEM accumulators of 2 x NT columns
constexpr int kPromoWarps = 4;
constexpr int kTmaWarp = 4;
constexpr int kMmaWarp = 5;
constexpr int kThreads = 6 * 32;
constexpr uint32_t kABytes = 2 * BW * BK;   // two weight blocks
constexpr uint32_t kBBytes = NT * BK;       // token codes
constexpr uint32_t kStageBytes = kABytes + kBBytes;  // 36 KB
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxKB = 64;        // K <= 8192
constexpr int kMaxExperts = 1024;
constexpr int kOutRowBytes = 2 * BW * 2 + 16;  // bf16 row of 256 outputs, padded
constexpr uint32_t kOutBytes = NT * kOutRowBytes;

struct DecodeParams {
  const float* a_scales;   // token scales [rows_total, KB]
  const float* b_scales;   // weight scales [E, N/128, KB]
  const int32_t* offsets;
  int rows_total;
  int kblocks;
  int N;
  int E;
  int n_pairs;             // block pairs per expert
  int I;
  int early_prefetch;
  uint16_t* out_bf16;
  float* out_f32;
  uint8_t* h_codes;
  float* h_scales;
  uint16_t* h_bf16;
  const int32_t* sorted_pair;
  const float* pair_weights;
  int* status;
  unsigned long long wait_limit_ns;
  int stop_after_stages;
};

// Scales of one tile: token scales transposed to [kb][token], the two weight-block scales per
// K-block, and (down) the combine weights of the tile's rows.
struct Slab {
  float sx[kMaxKB][NT];
  float sw[kMaxKB][2];
  float w[NT];
};

struct __align__(8) SmemTail {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t tmem_full[kAccBufs];
  uint64_t tmem_empty[kAccBufs];
  uint64_t teardown;
  uint32_t tmem_addr;
  int abort_flag;
  int32_t off[kMaxExperts + 1];
  int32_t prefix[kMaxExperts + 1];
};

constexpr size_t kSmemBytes = 1024 + static_cast<size_t>(kStages) * kStageBytes + kOutBytes + 2 * sizeof(Slab) + sizeof(SmemTail);
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, SmemTail* s, const DecodeParams& p) {
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
// whole warp: every lane polls, then the lanes vote (no split warp after a wait)
__device__ __forceinline__ bool warp_wait_or_abort(uint64_t* bar, uint32_t parity, SmemTail* s, const DecodeParams& p) {
  return __all_sync(0xFFFFFFFFu, wait_or_abort(bar, parity, s, p) ? 1 : 0) != 0;
}

__device__ __forceinline__ float silu_mul(float g, float u) {  // as in the wide kernel
  return __fdividef(g, 1.0f + __expf(-g)) * u;
}

__device__ __forceinline__ void cp_async_4(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// weight rows (lo block, hi block) of tile (e, pair j), and their scale block-rows
template <int MODE>
__device__ __forceinline__ void tile_blocks(const DecodeParams& p, int e, int j, int& row_lo, int& row_hi, int& nb_lo,
                                            int& nb_hi) {
  const int NB = p.N / BW;
  if (MODE == kModeGateUp) {
    nb_lo = j;
    nb_hi = j + p.I / BW;
  } else {
    nb_lo = 2 * j;
    nb_hi = min(2 * j + 1, NB - 1);  // a half past N re-reads the last block; its columns are never stored
  }
  row_lo = e * p.N + nb_lo * BW;
  row_hi = e * p.N + nb_hi * BW;
}

template <int MODE>
__global__ void __launch_bounds__(kThreads, 1)
gemm_decode_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                   const DecodeParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* out_tile = smem + static_cast<size_t>(kStages) * kStageBytes;
  Slab* slab = reinterpret_cast<Slab*>(out_tile + kOutBytes);
  SmemTail* s = reinterpret_cast<SmemTail*>(slab + 2);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

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
    mbar_init(&s->teardown, 1);
    s->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kTmaWarp && lane == 0) {
    prefetch_tensormap(&tm_x);
    prefetch_tensormap(&tm_w);
  }
  if (warp == kMmaWarp) {
    tmem_alloc(&s->tmem_addr, kTmemCols);
    tmem_relinquish();
  }
  if (warp == kTmaWarp && lane == 0 && p.early_prefetch > 0) {
    // The weights do not depend on the kernels before this one in the stream: pull this CTA's first
    // weight tiles into L2 before waiting for them.  Tile T is guessed as (expert T / n_pairs, pair
    // T % n_pairs), exact when every expert has one chunk; a wrong guess costs an unused L2 fill.
    for (int t = 0; t < p.early_prefetch; ++t) {
      const int T = blockIdx.x + t * gridDim.x;
      if (T >= p.E * p.n_pairs) break;
      int row_lo, row_hi, nb_lo, nb_hi;
      tile_blocks<MODE>(p, T / p.n_pairs, T % p.n_pairs, row_lo, row_hi, nb_lo, nb_hi);
      for (int kb = 0; kb < p.kblocks; ++kb) {
        tma_prefetch_2d(&tm_w, kb * BK, row_lo);
        tma_prefetch_2d(&tm_w, kb * BK, row_hi);
      }
    }
  }
  pdl_wait();
  build_tile_list(s->off, s->prefix, p.offsets, p.rows_total, p.E, NT, p.n_pairs);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = s->tmem_addr;
  const int total_tiles = s->prefix[p.E];
  const int num_ctas = gridDim.x;  // every SM streams: the tiles are small, the last round costs little
  const int first_tile = static_cast<int>(blockIdx.x) < num_ctas ? static_cast<int>(blockIdx.x) : total_tiles;
  const int KB = p.kblocks;
  const int NB = p.N / BW;

  if (warp == kTmaWarp) {
    // =============================== TMA producer =======================================
    if (lane == 0) {
      int stage = 0, armed_total = 0, cur_e = 0;
      uint32_t phase = 0, armed = 0, armed_parity = 0;
      bool ok = true;
      for (int T = first_tile; ok && T < total_tiles; T += num_ctas) {
        const TileCoord c = decode_tile(s->off, s->prefix, NT, T, cur_e);
        int row_lo, row_hi, nb_lo, nb_hi;
        tile_blocks<MODE>(p, c.e, c.n_tile, row_lo, row_hi, nb_lo, nb_hi);
        for (int kb = 0; kb < KB; ++kb) {
          if (p.stop_after_stages >= 0 && armed_total >= p.stop_after_stages) { ok = false; break; }
          ++armed_total;
          if (!wait_or_abort(&s->empty[stage], phase ^ 1, s, p)) { ok = false; break; }
          uint8_t* a_dst = smem + static_cast<size_t>(stage) * kStageBytes;
          mbar_arrive_expect_tx(&s->full[stage], kStageBytes);
          tma_load_2d(a_dst, &tm_w, &s->full[stage], kb * BK, row_lo);
          tma_load_2d(a_dst + kABytes / 2, &tm_w, &s->full[stage], kb * BK, row_hi);
          tma_load_2d(a_dst + kABytes, &tm_x, &s->full[stage], kb * BK, c.m0);
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
    // =============================== MMA issuer =========================================
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_e4m3_f32(BW, NT);
      int stage = 0, ks = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int T = first_tile; ok && T < total_tiles; T += num_ctas) {
        for (int kb = 0; kb < KB; ++kb) {
          if (!wait_or_abort(&s->tmem_empty[ks], acc_phase ^ 1, s, p)) { ok = false; break; }
          if (!wait_or_abort(&s->full[stage], phase, s, p)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(smem + static_cast<size_t>(stage) * kStageBytes);
          const uint64_t w_lo = umma_desc_k_sw128(a_addr), w_hi = umma_desc_k_sw128(a_addr + kABytes / 2);
          const uint64_t x_desc = umma_desc_k_sw128(a_addr + kABytes);
          const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(ks) * (2 * NT);
#pragma unroll
          for (int k4 = 0; k4 < BK / 32; ++k4)  // +32 bytes of K = +2 in the 16-byte address field
            umma_f8(d_tmem, w_lo + 2 * k4, x_desc + 2 * k4, idesc, k4 > 0 ? 1u : 0u);
#pragma unroll
          for (int k4 = 0; k4 < BK / 32; ++k4)
            umma_f8(d_tmem + NT, w_hi + 2 * k4, x_desc + 2 * k4, idesc, k4 > 0 ? 1u : 0u);
          umma_commit(&s->empty[stage]);
          umma_commit(&s->tmem_full[ks]);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
          if (++ks == kAccBufs) { ks = 0; acc_phase ^= 1; }
        }
      }
      if (!ok) {  // after an abort MMAs may still be executing: wait (bounded) before TMEM goes away
        umma_commit(&s->teardown);
        mbar_wait_bounded(&s->teardown, 0, 20000000ull);
      }
    }
  } else {
    // =============================== promotion + epilogue warps =========================
    const int wr = warp * 32 + lane;  // weight row within a block = TMEM lane
    const int pt = threadIdx.x;       // 0..127
    const uint32_t lane_addr = static_cast<uint32_t>(warp * 32) << 16;
    int ks = 0, cur_e = 0, sb = 0;
    uint32_t acc_phase = 0;
    bool ok = true;

    // asynchronous fill of slab `b` with the scales (and combine weights) of tile c
    auto fill_slab = [&](int b, const TileCoord& c) {
      Slab& sl = slab[b];
      int row_lo, row_hi, nb_lo, nb_hi;
      tile_blocks<MODE>(p, c.e, c.n_tile, row_lo, row_hi, nb_lo, nb_hi);
      for (int i = pt; i < KB * NT; i += kPromoWarps * 32) {
        const int t = i / KB, kb = i - t * KB;  // consecutive threads read consecutive floats of a row
        cp_async_4(&sl.sx[kb][t], p.a_scales + static_cast<int64_t>(min(c.m0 + t, p.rows_total - 1)) * KB + kb);
      }
      const float* swb = p.b_scales + static_cast<int64_t>(c.e) * NB * KB;
      for (int i = pt; i < 2 * KB; i += kPromoWarps * 32) {
        const int h = i / KB, kb = i - h * KB;
        cp_async_4(&sl.sw[kb][h], swb + static_cast<int64_t>(h ? nb_hi : nb_lo) * KB + kb);
      }
      if (MODE == kModeDown && pt < NT) cp_async_4(&sl.w[pt], p.pair_weights + min(c.m0 + pt, p.rows_total - 1));
    };

    int T = first_tile;
    if (T < total_tiles) {
      TileCoord c = decode_tile(s->off, s->prefix, NT, T, cur_e);
      fill_slab(0, c);
      for (;;) {
        const int Tn = T + num_ctas;
        const bool has_next = Tn < total_tiles;
        TileCoord cn = c;
        cp_async_wait_all();                     // this tile's slab (issued one tile ago) has landed ...
        named_bar_sync(1, kPromoWarps * 32);     // ... for every thread, and the previous tile's readers are done
        if (has_next) {
          cn = decode_tile(s->off, s->prefix, NT, Tn, cur_e);
          fill_slab(sb ^ 1, cn);                 // next tile's scales fly while this tile computes
        }
        const Slab& sl = slab[sb];
        const int rows = min(NT, c.m_end - c.m0);  // live token rows of this tile (>= 1)

        float acc_lo[NT], acc_hi[NT];
#pragma unroll
        for (int t = 0; t < NT; ++t) acc_lo[t] = acc_hi[t] = 0.0f;

        for (int kb = 0; kb < KB; ++kb) {
          if (!warp_wait_or_abort(&s->tmem_full[ks], acc_phase, s, p)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t t0 = tmem_base + lane_addr + static_cast<uint32_t>(ks) * (2 * NT);
          uint32_t vl[NT], vh[NT];
          tmem_ld_x32(t0, vl);
          tmem_ld_x32(t0 + NT, vh);
          tmem_ld_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&s->tmem_empty[ks]);  // both reads have landed: hand the accumulator back
          if (++ks == kAccBufs) { ks = 0; acc_phase ^= 1; }
          const float2 sw = *reinterpret_cast<const float2*>(sl.sw[kb]);
#pragma unroll
          for (int t4 = 0; t4 < NT; t4 += 4) {
            const float4 sx = *reinterpret_cast<const float4*>(&sl.sx[kb][t4]);  // same address in every lane: broadcast
            const float sxs[4] = {sx.x, sx.y, sx.z, sx.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              acc_lo[t4 + u] = __fmaf_rn(__fmul_rn(sxs[u], sw.x), __uint_as_float(vl[t4 + u]), acc_lo[t4 + u]);
              acc_hi[t4 + u] = __fmaf_rn(__fmul_rn(sxs[u], sw.y), __uint_as_float(vh[t4 + u]), acc_hi[t4 + u]);
            }
          }
        }
        if (!ok) break;

        // ---- epilogue: transpose through shared memory, finish per token row ----------------
        const int j = c.n_tile;
        if (MODE == kModeGateUp) {
          // h = bf16( silu(bf16 gate) * bf16 up ), this thread's column of the 128-wide group
          uint16_t* T16 = reinterpret_cast<uint16_t*>(out_tile);
#pragma unroll
          for (int t = 0; t < NT; ++t) {
            const uint32_t gb = f32_to_bf16_bits(acc_lo[t]), ub = f32_to_bf16_bits(acc_hi[t]);
            const uint32_t hb = f32_to_bf16_bits(silu_mul(bf16_bits_to_f32(gb), bf16_bits_to_f32(ub)));
            T16[t * (kOutRowBytes / 2) + wr] = static_cast<uint16_t>(hb);
            if (p.out_bf16 && t < rows) {  // debug dump of the bf16 gate_up row
              uint16_t* gd = p.out_bf16 + static_cast<int64_t>(c.m0 + t) * p.N + j * BW + wr;
              gd[0] = static_cast<uint16_t>(gb);
              gd[p.I] = static_cast<uint16_t>(ub);
            }
          }
          named_bar_sync(2, kPromoWarps * 32);
          const int IB = p.I / BW;
          for (int t = warp; t < rows; t += kPromoWarps) {  // a warp per token row, 4 columns per lane
            const uint2 hv = *reinterpret_cast<const uint2*>(out_tile + t * kOutRowBytes + lane * 8);
            uint32_t m = __vmaxu2(hv.x & 0x7FFF7FFFu, hv.y & 0x7FFF7FFFu);  // |bf16| bit patterns: exact, order-free max
            m = max(m & 0xFFFFu, m >> 16);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
            float inv;
            const float sc = block_scale(bf16_bits_to_f32(m), &inv);
            const uint32_t cw = cvt_e4m3x4(__fmul_rn(bf16_bits_to_f32(hv.x & 0xFFFFu), inv), __fmul_rn(__uint_as_float(hv.x & 0xFFFF0000u), inv),
                                           __fmul_rn(bf16_bits_to_f32(hv.y & 0xFFFFu), inv), __fmul_rn(__uint_as_float(hv.y & 0xFFFF0000u), inv));
            const int64_t row = c.m0 + t;
            *reinterpret_cast<uint32_t*>(p.h_codes + row * p.I + j * BW + lane * 4) = cw;
            if (lane == 0) p.h_scales[row * IB + j] = sc;
            if (p.h_bf16) *reinterpret_cast<uint2*>(p.h_bf16 + row * p.I + j * BW + lane * 4) = hv;
          }
        } else {
          const int col_lo = 2 * j * BW + wr, col_hi = col_lo + BW;
          const bool hi_ok = col_hi < p.N;
          uint16_t* T16 = reinterpret_cast<uint16_t*>(out_tile);
#pragma unroll
          for (int t = 0; t < NT; ++t) {
            float lo = acc_lo[t], hi = acc_hi[t];
            if (p.out_f32 && t < rows) {  // debug dump of the fp32 accumulators
              float* d = p.out_f32 + static_cast<int64_t>(c.m0 + t) * p.N;
              d[col_lo] = lo;
              if (hi_ok) d[col_hi] = hi;
            }
            if (MODE == kModeDown) {  // contribution = bf16( fl(w * y) )
              const float w = sl.w[t];
              lo = __fmul_rn(w, lo);
              hi = __fmul_rn(w, hi);
            }
            T16[t * (kOutRowBytes / 2) + wr] = static_cast<uint16_t>(f32_to_bf16_bits(lo));
            T16[t * (kOutRowBytes / 2) + BW + wr] = static_cast<uint16_t>(f32_to_bf16_bits(hi));
          }
          named_bar_sync(2, kPromoWarps * 32);
          for (int t = warp; t < rows; t += kPromoWarps) {  // a warp per output row: 512 bytes, 16 per lane
            const int row = c.m0 + t;
            int64_t out_row = row;
            if (MODE == kModeDown && p.sorted_pair) out_row = min(max(__ldg(p.sorted_pair + row), 0), p.rows_total - 1);
            const uint4 v = *reinterpret_cast<const uint4*>(out_tile + t * kOutRowBytes + lane * 16);
            const int col = 2 * j * BW + 8 * lane;
            if (col < p.N) *reinterpret_cast<uint4*>(p.out_bf16 + out_row * p.N + col) = v;
          }
        }
        if (!has_next) break;
        T = Tn;
        c = cn;
        sb ^= 1;
      }
    }
    cp_async_wait_all();
  }

  // ---- teardown ---------------------------------------------------------------------------
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

CUresult make_tmap(EncodeTiledFn encode, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols};
  const cuuint32_t box[2] = {BK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return encode(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

template <int MODE>
cudaError_t launch_mode(const Launch& L, const CUtensorMap& tx, const CUtensorMap& tw, const DecodeParams& p, int grid) {
  static std::atomic<bool> attr_set_dev[64];  // sticky per function and device; set idempotently
  std::atomic<bool>& attr_set = attr_set_dev[L.device & 63];
  if (!attr_set.load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_decode_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kSmemBytes));
    if (e != cudaSuccess) return e;
    attr_set.store(true, std::memory_order_release);
  }
  ++*L.launches;
  return launch_pdl(gemm_decode_kernel<MODE>, static_cast<unsigned>(grid), kThreads, kSmemBytes, L.stream, tx, tw, p);
}

}  // namespace

bool gemm_decode_applies(const GemmArgs& a) {
  // grouped calls whose groups average at most 32 rows (decode batches), K within the scale slab
  return a.offsets != nullptr && a.rows_total <= static_cast<int64_t>(NT) * a.E && a.K / BK <= kMaxKB;
}

cudaError_t launch_gemm_decode(const Launch& L, EncodeTiledFn encode, const GemmArgs& a, CUresult* cu_err) {
  *cu_err = CUDA_SUCCESS;
  if (a.rows_total == 0) return cudaSuccess;
  CUtensorMap tx, tw;
  CUresult r = make_tmap(encode, &tx, a.a_codes, static_cast<uint64_t>(a.rows_total), static_cast<uint64_t>(a.K), NT);
  if (r == CUDA_SUCCESS)
    r = make_tmap(encode, &tw, a.b_codes, static_cast<uint64_t>(a.E * a.N), static_cast<uint64_t>(a.K), BW);
  if (r != CUDA_SUCCESS) {
    *cu_err = r;
    return cudaErrorUnknown;
  }
  DecodeParams p{};
  p.a_scales = a.a_scales;
  p.b_scales = a.b_scales;
  p.offsets = a.offsets;
  p.rows_total = static_cast<int>(a.rows_total);
  p.kblocks = static_cast<int>(a.K / BK);
  p.N = static_cast<int>(a.N);
  p.E = static_cast<int>(a.E);
  p.I = static_cast<int>(a.N / 2);
  p.n_pairs = a.mode == kModeGateUp ? static_cast<int>(a.N / 2 / BW) : static_cast<int>((a.N + 2 * BW - 1) / (2 * BW));
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
  {
    const int64_t tile_bytes = static_cast<int64_t>(p.kblocks) * kABytes;
    const int64_t budget = 80ll << 20;  // stay well inside the 126 MB L2
    p.early_prefetch = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(3, budget / (tile_bytes * L.sm_count))));
  }
  // upper bound on the tile count (group sizes live on the device): each expert adds at most one partial chunk
  const int64_t chunks_max = a.rows_total / NT + a.E;
  const int grid = static_cast<int>(std::min<int64_t>(L.sm_count, chunks_max * p.n_pairs));
  switch (a.mode) {
    case kModeLinear: return launch_mode<kModeLinear>(L, tx, tw, p, grid);
    case kModeGateUp: return launch_mode<kModeGateUp>(L, tx, tw, p, grid);
    case kModeDown: return launch_mode<kModeDown>(L, tx, tw, p, grid);
  }
  return cudaErrorInvalidValue;
}

}  // namespace qarl
