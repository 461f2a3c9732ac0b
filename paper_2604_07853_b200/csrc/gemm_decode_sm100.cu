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
// CTA = 512 threads, 128 registers each: warps 0-7 promotion (two threads per weight row -- warps w
// and w + 4 read the same TMEM lanes, token columns 0-15 and 16-31 --, 2 x 16 accumulators each; at the
// end of a tile they round to bf16 -- down: after the multiplication by the pair's combine weight --
// and transpose the tile through shared memory), warps 8-11 epilogue (a warp per token row while the
// promotion warps run the next tile: gate_up = SwiGLU, 1x128 amax / scale / e4m3 codes; down / linear =
// whole-row stores), warp 12 TMA producer, warps 13 and 14 MMA issuers (one per weight block of the pair).
// Every barrier wait is bounded as in the wide kernel; an expired wait aborts the CTA cleanly.
//
// The whole decode-sized MoE layer also runs as ONE launch of this kernel (kModeLayer): the tile
// list holds the gate_up tiles and the down tiles of every expert, the down tiles of expert e
// kDepSlots experts after its gate_up tiles, so the weight stream never stops between the two
// projections; a down tile starts once a per-expert counter says the h rows it reads are written
// (release by the writers, acquire + proxy fence by the readers, every spin bounded); tiles are
// drawn from a counter (they differ in size), and a CTA that has run out of tiles draws tokens
// and sums each -- its k contributions in ascending expert id (the combine), read from L2 -- as
// soon as the down tiles of the token's experts are done.  Tile arithmetic, promotion chain and
// epilogues are the ones of the separate launches: the bytes are the same.
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
constexpr int kPromoWarps = 8;     // warps 0-7: TMEM lane quadrant = warp % 4, token half = warp / 4
constexpr int kEpiWarps = 4;       // warps 8-11
constexpr int kTmaWarp = 12;
constexpr int kMmaWarp = 13;        // and 14: one issuer per weight block of the pair; warp 15 idle
constexpr int kThreads = 16 * 32;
constexpr int NTH = NT / 2;        // token columns per promotion thread
// 512 threads: 128 registers each, which every role fits (a promotion thread holds 2 x 16 accumulators and
// 2 x 16 partial sums in flight); no re-allocation between warpgroups
constexpr uint32_t kABytes = 2 * BW * BK;   // two weight blocks
constexpr uint32_t kBBytes = NT * BK;       // token codes
constexpr uint32_t kStageBytes = kABytes + kBBytes;  // 36 KB
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxKB = 64;        // K <= 8192
constexpr int kMaxExperts = 1024;
constexpr int kOutRowBytes = 2 * BW * 2 + 16;  // bf16 row of 256 outputs, padded
constexpr uint32_t kOutBytes = NT * kOutRowBytes;
constexpr int kModeLayer = 3;     // gate_up tiles + down tiles + combine in one launch (this file only)
constexpr int kDepSlots = 64;     // the down tiles of expert e are listed with the gate_up tiles of expert e + kDepSlots
constexpr int kMaxTopK = 32;
constexpr int kSchedSlots = 4;    // layer: tile numbers the producer has drawn and the other roles have not yet read

// Operands of one projection: token-side scales [rows_total, KB], weight scales [E, N/128, KB].
struct Proj {
  const float* a_scales;
  const float* b_scales;
  int kblocks;
  int N;
  int n_pairs;             // block pairs per expert
};

struct DecodeParams {
  Proj pj[2];              // [0]: the call's projection (layer: gate_up); [1]: the layer's down projection
  const int32_t* offsets;
  int rows_total;
  int E;
  int I;
  int early_prefetch;
  uint16_t* out_rows;      // linear: y [M, N]; down: contributions [P, H]
  uint16_t* dump_gate_up;  // gate_up (debug): bf16 gate_up [P, 2I]
  float* out_f32;          // linear / down (debug): fp32 accumulators
  uint8_t* h_codes;
  float* h_scales;
  uint16_t* h_bf16;
  const int32_t* sorted_pair;
  const float* pair_weights;
  // the layer in one launch
  const int32_t* ids;          // [M, k]
  const int32_t* pos_of_pair;  // [M * k]
  uint16_t* y;                 // [M, H]
  int M, k;
  int* sync;                   // [0]: tiles handed out so far; [1 + e]: finished gate_up tiles of expert e;
                               // [1 + E + e]: finished down tiles of expert e; [1 + 2E]: tokens handed out (all zero on entry)
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
  uint64_t out_full;
  uint64_t out_empty;
  uint64_t teardown[2];
  uint64_t sched_full[kSchedSlots];
  uint64_t sched_empty[kSchedSlots];
  int sched_T[kSchedSlots];
  uint32_t tmem_addr;
  int abort_flag;
  int ready_flag;
  int peek_T;
  int token_T;
  int pad_;
  int32_t order[1][kMaxTopK];  // combine: contribution row of the rank-th smallest expert id of a token
  int32_t off[kMaxExperts + 1];
  int32_t prefix[kMaxExperts + kDepSlots + 1];
};

constexpr size_t kSmemBytes = 1024 + static_cast<size_t>(kStages) * kStageBytes + kOutBytes + 2 * sizeof(Slab) + sizeof(SmemTail);
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

// One unit of work: projection `mode` (kModeLinear / kModeGateUp / kModeDown), expert e, block
// pair j, token rows [m0, min(m0 + NT, m_end)).
struct Tile {
  int mode, e, j, m0, m_end;
};

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

// ---- counters in global memory that CTAs of one launch publish to one another (layer mode) -------
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_gpu_add(int* p, int v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// orders this thread's generic-proxy accesses to global memory with its TMA (async-proxy) accesses
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

// Bounded wait until *ctr >= target (acquire).  A counter only waits on tiles listed earlier, and a tile
// is only ever held by a CTA that is running (tiles are drawn, not pre-assigned: a CTA of the grid that
// has not been scheduled yet, e.g. behind another stream's kernel, holds none), so the wait ends whatever
// part of the grid is resident; the bound is for a broken run.
__device__ __forceinline__ bool counter_wait_or_abort(const int* ctr, int target, SmemTail* s, const DecodeParams& p) {
  if (ld_acquire_gpu(ctr) >= target) return true;
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 16; ++i) {
      if (ld_acquire_gpu(ctr) >= target) return true;
      __nanosleep(100);
    }
    if (*reinterpret_cast<volatile int*>(&s->abort_flag)) return false;
    if (globaltimer_ns() - t0 > p.wait_limit_ns) {
      set_status(p.status, QARL_ERR_DEVICE_TIMEOUT);
      *reinterpret_cast<volatile int*>(&s->abort_flag) = 1;
      return false;
    }
  }
}

__device__ __forceinline__ float silu_mul(float g, float u) {  // as in the wide kernel
  return __fdividef(g, 1.0f + __expf(-g)) * u;
}

__device__ __forceinline__ void cp_async_4(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ __forceinline__ int chunks_of(const int32_t* off, int e) { return (max(off[e + 1] - off[e], 0) + NT - 1) / NT; }

// which operand set a tile uses: the layer's down tiles use pj[1], everything else pj[0]
template <int MODE>
__device__ __forceinline__ int proj_of(int mode) { return (MODE == kModeLayer && mode == kModeDown) ? 1 : 0; }

// weight rows (lo block, hi block) of a tile, and their scale block-rows
template <int MODE>
__device__ __forceinline__ void tile_blocks(const DecodeParams& p, const Tile& t, int& row_lo, int& row_hi, int& nb_lo,
                                            int& nb_hi) {
  const int N = p.pj[proj_of<MODE>(t.mode)].N;
  const int NB = N / BW;
  if (t.mode == kModeGateUp) {
    nb_lo = t.j;
    nb_hi = t.j + p.I / BW;
  } else {
    nb_lo = 2 * t.j;
    nb_hi = min(2 * t.j + 1, NB - 1);  // a half past N re-reads the last block; its columns are never stored
  }
  row_lo = t.e * N + nb_lo * BW;
  row_hi = t.e * N + nb_hi * BW;
}

// Layer mode.  Slot s of the list holds the gate_up tiles of expert s (s < E) followed by the down
// tiles of expert s - D (s >= D), D = min(kDepSlots, E): E + D slots.  prefix[s] = tiles before slot s.
__device__ __forceinline__ void build_layer_list(int32_t* off, int32_t* prefix, const DecodeParams& p, int D) {
  for (int e = threadIdx.x; e <= p.E; e += blockDim.x)
    off[e] = p.offsets ? min(max(p.offsets[e], 0), p.rows_total) : (e == 0 ? 0 : p.rows_total);
  __syncthreads();
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x, S = p.E + D;
    int carry = 0;
    for (int base = 0; base < S; base += 32) {
      const int sl = base + lane;
      int v = 0;
      if (sl < S) {
        if (sl < p.E) v += chunks_of(off, sl) * p.pj[0].n_pairs;
        if (sl >= D) v += chunks_of(off, sl - D) * p.pj[1].n_pairs;
      }
      int inc = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += u;
      }
      if (sl < S) prefix[sl] = carry + inc - v;
      carry += __shfl_sync(0xFFFFFFFFu, inc, 31);
    }
    if (lane == 0) prefix[S] = carry;
  }
  __syncthreads();
}

// Tile T of the list (T ascending per caller: `cur` only moves forward).
template <int MODE>
__device__ __forceinline__ Tile tile_at(const SmemTail* s, const DecodeParams& p, int D, int T, int& cur) {
  Tile t;
  if constexpr (MODE != kModeLayer) {
    const TileCoord c = decode_tile(s->off, s->prefix, NT, T, cur);
    t.mode = MODE;
    t.e = c.e;
    t.j = c.n_tile;
    t.m0 = c.m0;
    t.m_end = c.m_end;
    return t;
  } else {
    while (T >= s->prefix[cur + 1]) ++cur;
    int local = T - s->prefix[cur];
    const int gt = cur < p.E ? chunks_of(s->off, cur) * p.pj[0].n_pairs : 0;
    if (local < gt) {
      t.mode = kModeGateUp;
      t.e = cur;
    } else {
      t.mode = kModeDown;
      t.e = cur - D;
      local -= gt;
    }
    const int ch = chunks_of(s->off, t.e);
    t.j = local / ch;
    t.m0 = s->off[t.e] + (local % ch) * NT;
    t.m_end = s->off[t.e + 1];
    return t;
  }
}

template <int MODE>
__global__ void __launch_bounds__(kThreads, 1)
gemm_decode_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                   const __grid_constant__ CUtensorMap tm_x2, const __grid_constant__ CUtensorMap tm_w2,
                   const DecodeParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* out_tile = smem + static_cast<size_t>(kStages) * kStageBytes;
  Slab* slab = reinterpret_cast<Slab*>(out_tile + kOutBytes);
  SmemTail* s = reinterpret_cast<SmemTail*>(slab + 2);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr bool kLayer = MODE == kModeLayer;
  const int D = kLayer ? min(kDepSlots, p.E) : 0;

  pdl_trigger();
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&s->full[i], 1);
      mbar_init(&s->empty[i], 2);      // the commits of the two MMA issuers
    }
    for (int i = 0; i < kAccBufs; ++i) {
      mbar_init(&s->tmem_full[i], 2);  // the two MMA issuers
      mbar_init(&s->tmem_empty[i], kPromoWarps);
    }
    mbar_init(&s->teardown[0], 1);
    mbar_init(&s->teardown[1], 1);
    for (int i = 0; i < kSchedSlots; ++i) {
      mbar_init(&s->sched_full[i], 1);
      mbar_init(&s->sched_empty[i], 2 + kPromoWarps + kEpiWarps);
    }
    mbar_init(&s->out_full, kPromoWarps);
    mbar_init(&s->out_empty, kEpiWarps);
    s->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kTmaWarp && lane == 0) {
    prefetch_tensormap(&tm_x);
    prefetch_tensormap(&tm_w);
    if (kLayer) {
      prefetch_tensormap(&tm_x2);
      prefetch_tensormap(&tm_w2);
    }
  }
  if (warp == kMmaWarp) {
    tmem_alloc(&s->tmem_addr, kTmemCols);
    tmem_relinquish();
  }
  if (warp == kTmaWarp && lane == 0 && p.early_prefetch > 0) {
    // The weights do not depend on the kernels before this one in the stream: pull this CTA's first
    // weight tiles into L2 before waiting for them.  Tile T is guessed as (expert T / n_pairs, pair
    // T % n_pairs) of the first projection, exact when every expert has one chunk (the layer's list
    // starts with gate_up tiles only); a wrong guess costs an unused L2 fill.
    for (int t = 0; t < p.early_prefetch; ++t) {
      const int T = blockIdx.x + t * gridDim.x;
      if (T >= p.E * p.pj[0].n_pairs) break;
      Tile g;
      g.mode = kLayer ? kModeGateUp : MODE;
      g.e = T / p.pj[0].n_pairs;
      g.j = T % p.pj[0].n_pairs;
      int row_lo, row_hi, nb_lo, nb_hi;
      tile_blocks<MODE>(p, g, row_lo, row_hi, nb_lo, nb_hi);
      const uint64_t stream_once = l2_policy_evict_first();
      for (int kb = 0; kb < p.pj[0].kblocks; ++kb) {
        tma_prefetch_2d_hint(&tm_w, kb * BK, row_lo, stream_once);
        tma_prefetch_2d_hint(&tm_w, kb * BK, row_hi, stream_once);
      }
    }
  }
  pdl_wait();
  if (kLayer) build_layer_list(s->off, s->prefix, p, D);
  else build_tile_list(s->off, s->prefix, p.offsets, p.rows_total, p.E, NT, p.pj[0].n_pairs);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = s->tmem_addr;
  const int total_tiles = s->prefix[kLayer ? p.E + D : p.E];
  // Which tiles a CTA runs.  Single projection: tile blockIdx.x, then every gridDim.x-th (every SM
  // streams: the tiles are equal and small, the last round costs little).  Layer: the tiles differ in
  // size (a gate_up tile streams 2.7 x the bytes of a down tile), so the CTAs draw tile numbers from a
  // counter in global memory as they go: the producer thread draws, the other roles read the numbers
  // from a small ring in shared memory in the same order.
  const int num_ctas = gridDim.x;
  const int first_tile = blockIdx.x;


  if (warp >= kPromoWarps + kEpiWarps) {
    if (warp == kTmaWarp) {
      // =============================== TMA producer =======================================
      if (lane == 0) {
        int stage = 0, armed_total = 0, cur = 0, sslot = 0;
        uint32_t phase = 0, armed = 0, armed_parity = 0, sphase = 0;
        bool ok = true;
        // The weights are read once per call: loaded with the evict-first policy they do not push the small
        // data the layer's kernels share through L2 (activations, codes, contributions) out of it.
        const uint64_t stream_once = l2_policy_evict_first();
        auto draw = [&](int prev) -> int {  // next tile of this CTA, -1: none
          if constexpr (!kLayer) {
            const int t = prev < 0 ? first_tile : prev + num_ctas;
            return t < total_tiles ? t : -1;
          } else {
            if (!wait_or_abort(&s->sched_empty[sslot], sphase ^ 1, s, p)) { ok = false; return -1; }
            int t = atomicAdd(p.sync, 1);
            if (t >= total_tiles) t = -1;
            *reinterpret_cast<volatile int*>(&s->sched_T[sslot]) = t;
            mbar_arrive(&s->sched_full[sslot]);  // release: the number is visible to whoever sees the phase flip
            if (++sslot == kSchedSlots) { sslot = 0; sphase ^= 1; }
            return t;
          }
        };
        for (int T = draw(-1); ok && T >= 0; T = draw(T)) {
          const Tile c = tile_at<MODE>(s, p, D, T, cur);
          const int pi = proj_of<MODE>(c.mode);
          int row_lo, row_hi, nb_lo, nb_hi;
          tile_blocks<MODE>(p, c, row_lo, row_hi, nb_lo, nb_hi);
          const CUtensorMap* mx = pi ? &tm_x2 : &tm_x;
          const CUtensorMap* mw = pi ? &tm_w2 : &tm_w;
          if (kLayer && c.mode == kModeDown) {
            // the h codes of this expert are written by gate_up tiles of this launch (other CTAs)
            if (!counter_wait_or_abort(p.sync + 1 + c.e, chunks_of(s->off, c.e) * p.pj[0].n_pairs, s, p)) { ok = false; break; }
            fence_proxy_async_global();
          }
          const int KB = p.pj[pi].kblocks;
          for (int kb = 0; kb < KB; ++kb) {
            if (p.stop_after_stages >= 0 && armed_total >= p.stop_after_stages) { ok = false; break; }
            ++armed_total;
            if (!wait_or_abort(&s->empty[stage], phase ^ 1, s, p)) { ok = false; break; }
            uint8_t* a_dst = smem + static_cast<size_t>(stage) * kStageBytes;
            mbar_arrive_expect_tx(&s->full[stage], kStageBytes);
            tma_load_2d_hint(a_dst, mw, &s->full[stage], kb * BK, row_lo, stream_once);
            tma_load_2d_hint(a_dst + kABytes / 2, mw, &s->full[stage], kb * BK, row_hi, stream_once);
            tma_load_2d(a_dst + kABytes, mx, &s->full[stage], kb * BK, c.m0);
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
      // =============================== MMA issuers ========================================
      // One thread per weight block of the pair: each feeds its own 32 columns of the accumulator, so the
      // two never write the same TMEM columns, and the fixed cost per K-block of waiting, issuing and
      // committing (which holds the shared-memory stage, i.e. bytes in flight from HBM) is halved.
      if (lane == 0) {
        const int half = warp - kMmaWarp;
        constexpr uint32_t idesc = umma_idesc_e4m3_f32(BW, NT);
        int stage = 0, ks = 0, cur = 0, sslot = 0;
        uint32_t phase = 0, acc_phase = 0, sphase = 0;
        bool ok = true;
        auto take = [&](int prev) -> int {
          if constexpr (!kLayer) {
            const int t = prev < 0 ? first_tile : prev + num_ctas;
            return t < total_tiles ? t : -1;
          } else {
            if (!wait_or_abort(&s->sched_full[sslot], sphase, s, p)) { ok = false; return -1; }
            const int t = *reinterpret_cast<volatile int*>(&s->sched_T[sslot]);
            mbar_arrive(&s->sched_empty[sslot]);
            if (++sslot == kSchedSlots) { sslot = 0; sphase ^= 1; }
            return t;
          }
        };
        for (int T = take(-1); ok && T >= 0; T = take(T)) {
          int KB = p.pj[0].kblocks;
          if (kLayer) KB = p.pj[proj_of<MODE>(tile_at<MODE>(s, p, D, T, cur).mode)].kblocks;
          for (int kb = 0; kb < KB; ++kb) {
            if (!wait_or_abort(&s->tmem_empty[ks], acc_phase ^ 1, s, p)) { ok = false; break; }
            if (!wait_or_abort(&s->full[stage], phase, s, p)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t a_addr = smem_u32(smem + static_cast<size_t>(stage) * kStageBytes);
            const uint64_t w_desc = umma_desc_k_sw128(a_addr + half * (kABytes / 2));
            const uint64_t x_desc = umma_desc_k_sw128(a_addr + kABytes);
            const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(ks) * (2 * NT) + static_cast<uint32_t>(half) * NT;
#pragma unroll
            for (int k4 = 0; k4 < BK / 32; ++k4)  // +32 bytes of K = +2 in the 16-byte address field
              umma_f8(d_tmem, w_desc + 2 * k4, x_desc + 2 * k4, idesc, k4 > 0 ? 1u : 0u);
            umma_commit(&s->empty[stage]);
            umma_commit(&s->tmem_full[ks]);
            if (++stage == kStages) { stage = 0; phase ^= 1; }
            if (++ks == kAccBufs) { ks = 0; acc_phase ^= 1; }
          }
        }
        if (!ok) {  // after an abort MMAs may still be executing: wait (bounded) before TMEM goes away
          umma_commit(&s->teardown[half]);
          mbar_wait_bounded(&s->teardown[half], 0, 20000000ull);
        }
      }
    }
  } else if (warp < kPromoWarps) {
    // =============================== promotion warps ====================================
    // Two threads per weight row: warps w and w + 4 read the same TMEM lanes, the first the partial sums
    // of token columns 0-15, the second those of columns 16-31 (of both weight blocks).
    const int wr = (warp & 3) * 32 + lane;  // weight row within a block = TMEM lane
    const int tb = (warp >> 2) * NTH;       // first token column of this thread
    const int pt = threadIdx.x;             // 0..255
    constexpr uint32_t kPromoThreads = kPromoWarps * 32;
    const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
    int ks = 0, cur = 0, sb = 0;
    uint32_t acc_phase = 0, tile_iter = 0;
    bool ok = true;

    // Fill of slab `b` with the scales (and combine weights) of tile c, asynchronous where the data
    // are inputs of the launch.  The h scales of a layer's down tile are written by other CTAs of this
    // launch: they are read (from L2) only once the expert's counter says they are complete.  With
    // `blocking` false an incomplete expert makes the call return at once with `filled` false -- a CTA
    // must never wait for a later tile's inputs while its current tile is unfinished (two CTAs could
    // then wait for each other's current tiles); the caller fills that slab when the tile is current.
    auto fill_slab = [&](int b, const Tile& c, bool blocking, bool& filled) -> bool {
      Slab& sl = slab[b];
      const Proj& pj = p.pj[proj_of<MODE>(c.mode)];
      const int KB = pj.kblocks, NB = pj.N / BW;
      filled = true;
      int row_lo, row_hi, nb_lo, nb_hi;
      tile_blocks<MODE>(p, c, row_lo, row_hi, nb_lo, nb_hi);
      if (kLayer && c.mode == kModeDown) {
        const int* ctr = p.sync + 1 + c.e;
        const int target = chunks_of(s->off, c.e) * p.pj[0].n_pairs;
        if (!blocking) {
          // one thread decides for all (threads reading the counter on their own could disagree)
          if (pt == 0) *reinterpret_cast<volatile int*>(&s->ready_flag) = ld_acquire_gpu(ctr) >= target ? 1 : 0;
          named_bar_sync(3, kPromoThreads);
          const int ready = *reinterpret_cast<volatile int*>(&s->ready_flag);
          named_bar_sync(3, kPromoThreads);
          if (!ready) { filled = false; return true; }
          (void)ld_acquire_gpu(ctr);  // every reading thread acquires
        } else if (!counter_wait_or_abort(ctr, target, s, p)) {
          return false;
        }
        for (int i = pt; i < KB * NT; i += kPromoThreads) {
          const int t = i / KB, kb = i - t * KB;
          sl.sx[kb][t] = __ldcg(pj.a_scales + static_cast<int64_t>(min(c.m0 + t, p.rows_total - 1)) * KB + kb);
        }
      } else {
        for (int i = pt; i < KB * NT; i += kPromoThreads) {
          const int t = i / KB, kb = i - t * KB;  // consecutive threads read consecutive floats of a row
          cp_async_4(&sl.sx[kb][t], pj.a_scales + static_cast<int64_t>(min(c.m0 + t, p.rows_total - 1)) * KB + kb);
        }
      }
      const float* swb = pj.b_scales + static_cast<int64_t>(c.e) * NB * KB;
      for (int i = pt; i < 2 * KB; i += kPromoThreads) {
        const int h = i / KB, kb = i - h * KB;
        cp_async_4(&sl.sw[kb][h], swb + static_cast<int64_t>(h ? nb_hi : nb_lo) * KB + kb);
      }
      if (c.mode == kModeDown && pt < NT) cp_async_4(&sl.w[pt], p.pair_weights + min(c.m0 + pt, p.rows_total - 1));
      return true;
    };

    int sslot = 0;
    uint32_t sphase = 0;
    // Next tile number of this CTA for all 128 threads (-1: none).  Layer: waits for the producer's
    // next draw; the four warps then agree on whether all of them got it.
    auto take = [&](int prev) -> int {
      if constexpr (!kLayer) {
        const int t = prev < 0 ? first_tile : prev + num_ctas;
        return t < total_tiles ? t : -1;
      } else {
        const bool got = warp_wait_or_abort(&s->sched_full[sslot], sphase, s, p);
        const int t = *reinterpret_cast<volatile int*>(&s->sched_T[sslot]);
        __syncwarp();
        if (got && lane == 0) mbar_arrive(&s->sched_empty[sslot]);
        if (++sslot == kSchedSlots) { sslot = 0; sphase ^= 1; }
        if (!named_bar_all(3, kPromoThreads, got)) { ok = false; return -1; }
        return t;
      }
    };

    // The four warps take every branch that holds a barrier together: `ok` is agreed on at the top
    // of a tile, and a warp whose wait ran out inside a tile skips the work but not the barriers.
    int T = take(-1);
    if (T >= 0) {
      Tile c = tile_at<MODE>(s, p, D, T, cur);
      bool filled = false;  // is the current tile's slab on its way?
      for (;;) {
        if (!filled) ok = fill_slab(sb, c, true, filled) && ok;
        Tile cn = c;
        cp_async_wait_all();                       // this tile's slab has landed ...
        ok = named_bar_all(1, kPromoThreads, ok);  // ... for every thread, and the previous tile's readers are done
        if (!ok) break;
        // the tile after this one: -1 none, -2 not drawn yet (layer only; taken at the end of this tile)
        int Tn;
        if constexpr (!kLayer) {
          Tn = T + num_ctas < total_tiles ? T + num_ctas : -1;
        } else {
          if (pt == 0)
            *reinterpret_cast<volatile int*>(&s->peek_T) =
                mbar_try_wait(&s->sched_full[sslot], sphase) ? *reinterpret_cast<volatile int*>(&s->sched_T[sslot]) : -2;
          named_bar_sync(3, kPromoThreads);  // one thread looks for all: the four warps must take the same branch
          Tn = *reinterpret_cast<volatile int*>(&s->peek_T);
          if (Tn != -2) {
            if (lane == 0) mbar_arrive(&s->sched_empty[sslot]);
            if (++sslot == kSchedSlots) { sslot = 0; sphase ^= 1; }
          }
        }
        bool next_filled = false;
        if (Tn >= 0) {
          cn = tile_at<MODE>(s, p, D, Tn, cur);
          fill_slab(sb ^ 1, cn, false, next_filled);  // next tile's scales fly while this tile computes
        }
        const Slab& sl = slab[sb];
        const int rows = min(NT, c.m_end - c.m0);  // live token rows of this tile (>= 1)
        const int pi = proj_of<MODE>(c.mode);
        const int KB = p.pj[pi].kblocks, N = p.pj[pi].N;

        float acc_lo[NTH], acc_hi[NTH];
#pragma unroll
        for (int t = 0; t < NTH; ++t) acc_lo[t] = acc_hi[t] = 0.0f;

        for (int kb = 0; kb < KB; ++kb) {
          if (!warp_wait_or_abort(&s->tmem_full[ks], acc_phase, s, p)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t t0 = tmem_base + lane_addr + static_cast<uint32_t>(ks) * (2 * NT) + static_cast<uint32_t>(tb);
          uint32_t vl[NTH], vh[NTH];
          tmem_ld_x16(t0, vl);
          tmem_ld_x16(t0 + NT, vh);
          tmem_ld_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&s->tmem_empty[ks]);  // both reads have landed: hand the accumulator back
          if (++ks == kAccBufs) { ks = 0; acc_phase ^= 1; }
          const float2 sw = *reinterpret_cast<const float2*>(sl.sw[kb]);
#pragma unroll
          for (int t4 = 0; t4 < NTH; t4 += 4) {
            const float4 sx = *reinterpret_cast<const float4*>(&sl.sx[kb][tb + t4]);  // same address in every lane: broadcast
            const float sxs[4] = {sx.x, sx.y, sx.z, sx.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              acc_lo[t4 + u] = __fmaf_rn(__fmul_rn(sxs[u], sw.x), __uint_as_float(vl[t4 + u]), acc_lo[t4 + u]);
              acc_hi[t4 + u] = __fmaf_rn(__fmul_rn(sxs[u], sw.y), __uint_as_float(vh[t4 + u]), acc_hi[t4 + u]);
            }
          }
        }

        // ---- hand the tile to the epilogue warps: bf16, transposed to [token][256 weight rows] ----
        if (ok && c.mode != kModeGateUp && p.out_f32) {  // debug dump of the fp32 accumulators
          const int col_lo = 2 * c.j * BW + wr, col_hi = col_lo + BW;
#pragma unroll
          for (int t = 0; t < NTH; ++t) {
            if (tb + t < rows) {
              float* d = p.out_f32 + static_cast<int64_t>(c.m0 + tb + t) * N;
              d[col_lo] = acc_lo[t];
              if (col_hi < N) d[col_hi] = acc_hi[t];
            }
          }
        }
        if (ok) ok = warp_wait_or_abort(&s->out_empty, (tile_iter & 1u) ^ 1u, s, p);  // previous tile drained
        if (ok) {
          uint16_t* T16 = reinterpret_cast<uint16_t*>(out_tile);
#pragma unroll
          for (int t = 0; t < NTH; ++t) {
            float lo = acc_lo[t], hi = acc_hi[t];
            if (c.mode == kModeDown) {  // contribution = bf16( fl(w * y) )
              const float w = sl.w[tb + t];
              lo = __fmul_rn(w, lo);
              hi = __fmul_rn(w, hi);
            }
            T16[(tb + t) * (kOutRowBytes / 2) + wr] = static_cast<uint16_t>(f32_to_bf16_bits(lo));
            T16[(tb + t) * (kOutRowBytes / 2) + BW + wr] = static_cast<uint16_t>(f32_to_bf16_bits(hi));
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&s->out_full);  // release: the epilogue warps see the tile after their wait
        }
        ++tile_iter;
        if (kLayer && Tn == -2) {  // the producer had not drawn the next tile when this one began: wait for it now
          Tn = take(T);
          if (Tn >= 0) cn = tile_at<MODE>(s, p, D, Tn, cur);
        }
        if (Tn < 0) break;
        T = Tn;
        c = cn;
        sb ^= 1;
        filled = next_filled;
      }
    }
    cp_async_wait_all();
  } else {
    // =============================== epilogue warps =====================================
    // They finish the staged bf16 tile per token row while the promotion warps are already in the
    // next tile: gate_up = SwiGLU, 1x128 amax / scale / e4m3 codes; down / linear = row stores.
    const int ew = warp - kPromoWarps;
    const int et = threadIdx.x - kPromoWarps * 32;  // 0..127 (the epilogue's threads)
    constexpr uint32_t kEpiThreads = kEpiWarps * 32;
    int cur = 0, sslot = 0;
    uint32_t sphase = 0, tile_iter = 0;
    bool ok = true;
    auto take = [&](int prev) -> int {
      if constexpr (!kLayer) {
        const int t = prev < 0 ? first_tile : prev + num_ctas;
        return t < total_tiles ? t : -1;
      } else {
        if (!warp_wait_or_abort(&s->sched_full[sslot], sphase, s, p)) { ok = false; return -1; }
        const int t = *reinterpret_cast<volatile int*>(&s->sched_T[sslot]);
        __syncwarp();
        if (lane == 0) mbar_arrive(&s->sched_empty[sslot]);
        if (++sslot == kSchedSlots) { sslot = 0; sphase ^= 1; }
        return t;
      }
    };
    for (int T = take(-1); T >= 0; T = take(T), ++tile_iter) {
      const Tile c = tile_at<MODE>(s, p, D, T, cur);
      const int rows = min(NT, c.m_end - c.m0);
      const int N = p.pj[proj_of<MODE>(c.mode)].N;
      const int j = c.j;
      ok = warp_wait_or_abort(&s->out_full, tile_iter & 1u, s, p);
      if (kLayer) ok = named_bar_all(4, kEpiThreads, ok);  // the publish below has a barrier: one decision for the four warps
      if (!ok) break;
      if (c.mode == kModeGateUp) {
        const int IB = p.I / BW;
        for (int t = ew; t < rows; t += kEpiWarps) {  // a warp per token row, 4 columns per lane
          const uint2 gv = *reinterpret_cast<const uint2*>(out_tile + t * kOutRowBytes + lane * 8);
          const uint2 uv = *reinterpret_cast<const uint2*>(out_tile + t * kOutRowBytes + BW * 2 + lane * 8);
          // h = bf16( silu(bf16 gate) * bf16 up )
          uint2 hv;
          hv.x = pack_bf16x2(silu_mul(bf16_bits_to_f32(gv.x & 0xFFFFu), bf16_bits_to_f32(uv.x & 0xFFFFu)),
                             silu_mul(__uint_as_float(gv.x & 0xFFFF0000u), __uint_as_float(uv.x & 0xFFFF0000u)));
          hv.y = pack_bf16x2(silu_mul(bf16_bits_to_f32(gv.y & 0xFFFFu), bf16_bits_to_f32(uv.y & 0xFFFFu)),
                             silu_mul(__uint_as_float(gv.y & 0xFFFF0000u), __uint_as_float(uv.y & 0xFFFF0000u)));
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
          if (p.dump_gate_up) {  // debug dump of the bf16 gate_up row
            uint16_t* gd = p.dump_gate_up + row * N + j * BW + lane * 4;
            *reinterpret_cast<uint2*>(gd) = gv;
            *reinterpret_cast<uint2*>(gd + p.I) = uv;
          }
        }
      } else {
        for (int t = ew; t < rows; t += kEpiWarps) {  // a warp per output row: 512 bytes, 16 per lane
          const int row = c.m0 + t;
          int64_t out_row = row;
          if (c.mode == kModeDown && p.sorted_pair) out_row = min(max(__ldg(p.sorted_pair + row), 0), p.rows_total - 1);
          const uint4 v = *reinterpret_cast<const uint4*>(out_tile + t * kOutRowBytes + lane * 16);
          const int col = 2 * j * BW + 8 * lane;
          if (col < N) *reinterpret_cast<uint4*>(p.out_rows + out_row * N + col) = v;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&s->out_empty);  // the staging tile may be overwritten
      if (kLayer) {
        // Other CTAs read what this tile wrote once the expert's counter says so -- the h codes by TMA
        // and their scales by plain loads (gate_up), the contribution rows in the k-sum (down): every
        // writer orders its stores (both proxies), then one thread bumps the counter.
        __threadfence();
        if (c.mode == kModeGateUp) fence_proxy_async_global();
        named_bar_sync(4, kEpiThreads);
        if (et == 0) red_release_gpu_add(p.sync + (c.mode == kModeGateUp ? 1 : 1 + p.E) + c.e, 1);
      }
    }

    if (kLayer) {
      // ---- the combine --------------------------------------------------------------------------
      // out[t] = bf16( sum of the token's k bf16 contributions in ascending expert id, from 0.0f ).
      // A CTA that has run out of tiles draws tokens from a counter and sums each as soon as the down tiles
      // of the token's k experts are all finished (their counters), while others still stream.
      ok = named_bar_all(4, kEpiThreads, ok);
      const int k = p.k, H = p.pj[1].N;
      const int64_t P = static_cast<int64_t>(p.M) * k;
      const int* dcount = p.sync + 1 + p.E;
      if (ok) {
        for (;;) {
          // tokens are drawn like tiles: the CTAs that run out of tiles first sum the most tokens
          if (et == 0) *reinterpret_cast<volatile int*>(&s->token_T) = atomicAdd(p.sync + 1 + 2 * p.E, 1);
          named_bar_sync(4, kEpiThreads);
          const int64_t t = *reinterpret_cast<volatile int*>(&s->token_T);
          if (t >= p.M) break;
          // lane l < k of every warp holds the token's l-th pair: its rank among the token's expert ids
          // gives the position of its row in the sum; the lane also waits for its expert's down tiles
          const int mine = lane < k ? p.ids[t * k + lane] : 0x7FFFFFFF;
          const int64_t pos = lane < k ? p.pos_of_pair[t * k + lane] : 0;
          int rank = 0;
          bool repeated = false;
          for (int jj = 0; jj < k; ++jj) {
            const int other = __shfl_sync(0xFFFFFFFFu, mine, jj);
            if (other < mine || (other == mine && jj < lane)) ++rank;
            if (other == mine && jj != lane) repeated = true;
          }
          named_bar_sync(4, kEpiThreads);  // the previous token's readers of order[] are done
          bool ready = true;
          if (lane < k) {
            if (ew == 0) {
              if (repeated) set_status(p.status, QARL_ERR_BAD_EXPERT_ID);  // expert repeated in a token
              s->order[0][rank] = static_cast<int32_t>(min(max(pos, int64_t(0)), P - 1));
            }
            if (mine >= 0 && mine < p.E)  // (a bad id has no row of its own: nothing to wait for)
              ready = counter_wait_or_abort(dcount + mine, chunks_of(s->off, mine) * p.pj[1].n_pairs, s, p);
          }
          ok = named_bar_all(4, kEpiThreads, ready);  // every warp has acquired; order[] is published
          if (!ok) break;
          const int32_t* ord = s->order[0];
          for (int col = et * 8; col < H; col += kEpiThreads * 8) {
            float acc[8];
#pragma unroll
            for (int i8 = 0; i8 < 8; ++i8) acc[i8] = 0.0f;
            for (int a0 = 0; a0 < k; a0 += 8) {  // eight rows' loads in flight, then the adds in rank order
              uint4 v[8];
#pragma unroll
              for (int a = 0; a < 8; ++a)
                v[a] = a0 + a < k ? __ldcg(reinterpret_cast<const uint4*>(p.out_rows + static_cast<int64_t>(ord[a0 + a]) * H + col))
                                  : make_uint4(0, 0, 0, 0);
#pragma unroll
              for (int a = 0; a < 8; ++a) {
                if (a0 + a < k) {
                  const uint32_t w[4] = {v[a].x, v[a].y, v[a].z, v[a].w};
#pragma unroll
                  for (int i4 = 0; i4 < 4; ++i4) {
                    acc[2 * i4] = __fadd_rn(acc[2 * i4], bf16_bits_to_f32(w[i4] & 0xFFFFu));
                    acc[2 * i4 + 1] = __fadd_rn(acc[2 * i4 + 1], bf16_bits_to_f32(w[i4] >> 16));
                  }
                }
              }
            }
            uint4 o;
            o.x = pack_bf16x2(acc[0], acc[1]);
            o.y = pack_bf16x2(acc[2], acc[3]);
            o.z = pack_bf16x2(acc[4], acc[5]);
            o.w = pack_bf16x2(acc[6], acc[7]);
            *reinterpret_cast<uint4*>(p.y + t * H + col) = o;
          }
        }
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
cudaError_t launch_mode(const Launch& L, const CUtensorMap& tx, const CUtensorMap& tw, const CUtensorMap& tx2,
                        const CUtensorMap& tw2, const DecodeParams& p, int grid) {
  static std::atomic<bool> attr_set_dev[64];  // sticky per function and device; set idempotently
  std::atomic<bool>& attr_set = attr_set_dev[L.device & 63];
  if (!attr_set.load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_decode_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kSmemBytes));
    if (e != cudaSuccess) return e;
    attr_set.store(true, std::memory_order_release);
  }
  ++*L.launches;
  return launch_pdl(gemm_decode_kernel<MODE>, static_cast<unsigned>(grid), kThreads, kSmemBytes, L.stream, tx, tw, tx2, tw2, p);
}

Proj make_proj(const GemmArgs& a) {
  Proj j{};
  j.a_scales = a.a_scales;
  j.b_scales = a.b_scales;
  j.kblocks = static_cast<int>(a.K / BK);
  j.N = static_cast<int>(a.N);
  j.n_pairs = a.mode == kModeGateUp ? static_cast<int>(a.N / 2 / BW) : static_cast<int>((a.N + 2 * BW - 1) / (2 * BW));
  return j;
}

// weight tiles a CTA pulls into L2 before the dependency wait (see the kernel)
int early_prefetch_tiles(const Launch& L, int kblocks) {
  const int64_t tile_bytes = static_cast<int64_t>(kblocks) * kABytes;
  const int64_t budget = 80ll << 20;  // stay well inside the 126 MB L2
  return static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(3, budget / (tile_bytes * L.sm_count))));
}

}  // namespace

bool gemm_decode_applies(const GemmArgs& a) {
  // grouped calls whose groups average at most 32 rows (decode batches) and dense calls of at most 64 rows
  // (a decode step's projections: more CTAs stream the weight, none multiplies padding); K within the scale slab
  if (a.K / BK > kMaxKB) return false;
  if (a.offsets == nullptr) return a.E == 1 && a.rows_total <= 2 * NT;
  return a.rows_total <= static_cast<int64_t>(NT) * a.E;
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
  p.pj[0] = make_proj(a);
  p.offsets = a.offsets;
  p.rows_total = static_cast<int>(a.rows_total);
  p.E = static_cast<int>(a.E);
  p.I = static_cast<int>(a.N / 2);
  if (a.mode == kModeGateUp) p.dump_gate_up = a.out_bf16;
  else p.out_rows = a.out_bf16;
  p.out_f32 = a.out_f32;
  p.h_codes = a.h_codes;
  p.h_scales = a.h_scales;
  p.h_bf16 = a.h_bf16;
  p.sorted_pair = a.sorted_pair;
  p.pair_weights = a.pair_weights;
  p.status = L.d_status;
  p.wait_limit_ns = L.wait_limit_ns ? L.wait_limit_ns : 2000000000ull;
  p.stop_after_stages = L.stop_after_stages;
  p.early_prefetch = early_prefetch_tiles(L, p.pj[0].kblocks);
  // upper bound on the tile count (group sizes live on the device): each expert adds at most one partial chunk
  const int64_t chunks_max = a.rows_total / NT + a.E;
  const int grid = static_cast<int>(std::min<int64_t>(L.sm_count, chunks_max * p.pj[0].n_pairs));
  switch (a.mode) {
    case kModeLinear: return launch_mode<kModeLinear>(L, tx, tw, tx, tw, p, grid);
    case kModeGateUp: return launch_mode<kModeGateUp>(L, tx, tw, tx, tw, p, grid);
    case kModeDown: return launch_mode<kModeDown>(L, tx, tw, tx, tw, p, grid);
  }
  return cudaErrorInvalidValue;
}

bool moe_decode_layer_applies(const GemmArgs& gate_up, const GemmArgs& down) {
  return gemm_decode_applies(gate_up) && gemm_decode_applies(down);
}

cudaError_t launch_moe_decode_layer(const Launch& L, EncodeTiledFn encode, const GemmArgs& g, const GemmArgs& d,
                                    const int32_t* ids, const int32_t* pos_of_pair, int64_t M, int64_t k, uint16_t* y,
                                    int* sync, CUresult* cu_err) {
  *cu_err = CUDA_SUCCESS;
  if (g.rows_total == 0) return cudaSuccess;
  CUtensorMap tx, tw, tx2, tw2;
  CUresult r = make_tmap(encode, &tx, g.a_codes, static_cast<uint64_t>(g.rows_total), static_cast<uint64_t>(g.K), NT);
  if (r == CUDA_SUCCESS) r = make_tmap(encode, &tw, g.b_codes, static_cast<uint64_t>(g.E * g.N), static_cast<uint64_t>(g.K), BW);
  if (r == CUDA_SUCCESS) r = make_tmap(encode, &tx2, d.a_codes, static_cast<uint64_t>(d.rows_total), static_cast<uint64_t>(d.K), NT);
  if (r == CUDA_SUCCESS) r = make_tmap(encode, &tw2, d.b_codes, static_cast<uint64_t>(d.E * d.N), static_cast<uint64_t>(d.K), BW);
  if (r != CUDA_SUCCESS) {
    *cu_err = r;
    return cudaErrorUnknown;
  }
  DecodeParams p{};
  p.pj[0] = make_proj(g);
  p.pj[1] = make_proj(d);
  p.offsets = g.offsets;
  p.rows_total = static_cast<int>(g.rows_total);
  p.E = static_cast<int>(g.E);
  p.I = static_cast<int>(g.N / 2);
  p.dump_gate_up = g.out_bf16;
  p.out_rows = d.out_bf16;
  p.out_f32 = d.out_f32;
  p.h_codes = g.h_codes;
  p.h_scales = g.h_scales;
  p.h_bf16 = g.h_bf16;
  p.sorted_pair = d.sorted_pair;
  p.pair_weights = d.pair_weights;
  p.ids = ids;
  p.pos_of_pair = pos_of_pair;
  p.y = y;
  p.M = static_cast<int>(M);
  p.k = static_cast<int>(k);
  p.sync = sync;
  p.status = L.d_status;
  p.wait_limit_ns = L.wait_limit_ns ? L.wait_limit_ns : 2000000000ull;
  p.stop_after_stages = L.stop_after_stages;
  p.early_prefetch = early_prefetch_tiles(L, p.pj[0].kblocks);
  // every SM takes part: the CTAs share the combine even when the tiles are few
  return launch_mode<kModeLayer>(L, tx, tw, tx2, tw2, p, L.sm_count);
}

}  // namespace qarl
