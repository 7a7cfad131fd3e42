// The whole layer stack of one verification round as ONE persistent kernel (sm_100a), one CTA per SM.
//
// A round is a chain of dependent steps per layer (RMSNorm -> QKV projection -> rotary + cache append -> tree
// attention -> merge of the key blocks -> O projection -> RMSNorm -> gate/up projection with SiLU * up -> down
// projection) followed by the final norm and the vocabulary projection with arg-max.  Run as separate kernels,
// every step pays a drain of the GPU, a launch, and a refill of the weight pipeline, and HBM idles meanwhile;
// at 64 tree tokens that was more than half of the time of a layer.  Here the CTAs stay resident for the whole
// stack:
//   * warp 0 streams weight tiles (TMA, 128-byte swizzle) into a shared-memory ring and never waits for
//     anything but a free ring slot, so the next projection's first tiles arrive while the small steps run;
//   * warp 10 fetches the matching activation blocks (hi / lo bf16 planes) once the step that produces them
//     has finished on every CTA, and is the TMA producer of the attention step;
//   * one thread of warp 1 issues every tcgen05.mma (projections: weights as the A operand, tokens as N, both
//     planes in one MMA of N = 2 x tokens; attention: S = Q K^T and O = P V as three hi/lo terms each);
//   * warps 2..9 drain TMEM (projection epilogues, softmax) and run the element-wise steps.
// Steps are separated by a grid-wide arrival counter in global memory instead of kernel boundaries: a CTA
// adds one when its part of a step is written, and whoever needs the step's output polls the counter (the
// activation producer for the projections' inputs, the worker warps for the element-wise steps).  The launch is
// cooperative, so all CTAs are co-resident; every wait is bounded by wall-clock time and ends the call with
// SPECASR_ERR_TIMEOUT in the status word instead of hanging.
//
// Work split.  Linear projections (QKV, O, down): weight tiles x k-parts, one CTA each; fp32 partial planes
// that the consuming step adds in plane order.  Non-linear epilogues (SiLU * up, arg-max): the (tile, k-block)
// list is cut into equal contiguous ranges, a tile that straddles two ranges is completed through a parked
// partial and a flag, in CTA order.  All of this is independent of timing, so results are deterministic.
//
// RMSNorm is split in two: the norm step adds the previous projection's planes to the residual stream,
// writes x * gain as hi / lo planes and leaves the row's sums of squares (two fixed halves per row); the
// consumer of the projection multiplies by rsqrt(mean(x^2) + eps), which commutes with the projection.  That
// removes the row-wide reduction from the path between two projections.
//
// The attention step borrows the ring's shared memory (Q / P tiles and K / V pages of one key block), so the
// weight producer resumes when the CTA's attention units are done.
#include "internal.h"
#include "device_utils.cuh"
#include "sm100_ptx.cuh"

using namespace sm100;

namespace {

constexpr int TILE_M = 128;
constexpr int SUB_K = 64;               // bf16 elements = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
#ifndef STACK_TM
#define STACK_TM 1
#endif
#ifndef STACK_KSUB
#define STACK_KSUB 2
#endif
// A ring stage holds TM weight tiles (128 rows each) of KSUB 64-wide k sub-blocks and ONE activation block that all
// of them multiply.  One tile of two sub-blocks (32 KB of weights, contiguous in the tile-packed layout) is what is
// built.  A tile pair of one sub-block (TM 2, KSUB 1) halves the activation bytes that cross from L2 into shared
// memory per weight byte, but doubles the k-parts and parked partial sums; it measured 7 % slower at 64 tokens and
// at 16, and leaving the activation loads out altogether shortens the call by 5 % only: they are not what bounds it.
constexpr int TM = STACK_TM;
constexpr int KSUB = STACK_KSUB;
constexpr int W_SUB_BYTES = TILE_M * SUB_K * 2;
constexpr int W_STAGE_BYTES = TM * KSUB * W_SUB_BYTES;
constexpr int MAX_STAGES = 6;
constexpr int SMEM_LIMIT = 227 * 1024;
constexpr int WORKERS = 256;            // warps 2..9
constexpr int NUM_THREADS = 352;        // + TMA weights, MMA, TMA activations
constexpr int NORM_PARTS = 2;           // fixed halves of a row whose sums of squares are kept apart

constexpr int KEYS_MAX = 208;           // cache positions per attention unit (13 pages of 16)
constexpr int ROUND = 128;              // keys whose probabilities fit the P tile at once
constexpr int SUB = 128 * 64 * 2;       // [128 rows][64 bf16] swizzled sub-tile (Q, P)
constexpr int KVSUB = KEYS_MAX * 64 * 2;

// steps of a layer, in order; step k of the call has its own arrival counter, complete when it equals the CTA count
// (one shared counter would not do: a CTA without work in a step runs ahead and would be counted for a later one)
enum { ST_NORM1 = 0, ST_QKV, ST_ROPE, ST_ATTN, ST_MERGE, ST_O, ST_NORM2, ST_GU, ST_DOWN, ST_PER_LAYER };

struct alignas(16) StackCtl {
  unsigned long long full[MAX_STAGES];
  unsigned long long empty[MAX_STAGES];
  unsigned long long acc_full[2];
  unsigned long long acc_empty[2];
  unsigned long long bar_qk, bar_v, bar_s, bar_p[2], bar_o[2];
  unsigned long long key[64];
  unsigned long long k1q[4][64], k2q[4][64];   // per lane quadrant: best and second-best packed key of a vocabulary tile
  float2 msq[4][64];                    // per lane quadrant: (max, sum of exp(x - max)) over the tile's rows
  float red_max[2][128];
  float red_sum[2][128];
  float inv[64];                        // 1 / rms of every token row, for the epilogue in progress
  float red[8];
  uint32_t tmem_base;
  int abort;
  int attn_done;                        // attention steps this CTA has finished (its ring memory is free again)
  int step_ok;                          // verdict of a wait that one worker made for all of them
  int units_done;                       // attention units the workers have finished (their shared memory is free again)
};

struct StackParams {
  int n_layers, d, qkv_dim, q_dim, Hq, Hkv, ffn, vocab, page_size, max_positions;
  float eps, scale_log2;
  const CUtensorMap* w_maps;            // [4 * n_layers + 1]: QKV, O, gate/up, down per layer, then the vocabulary
  const float* const* gains;            // [2 * n_layers + 1]: attention / FFN norm per layer, then the final norm
  const float2* rope;
  int n, n_pad, n_alloc, stages, stage_bytes, ring_bytes;
  int splits_qkv, splits_o, splits_down, epoch0, want_head, group, nodes_per_tile, row_tiles, attn_units;
  int32_t* ctl;                         // control block whose status word ends the call
  int32_t* sync;                        // [steps of the call] arrival counters, zeroed before the launch
  float* X;
  float* P;
  float* fixP;
  int32_t* fixFlag;
  bf16* H;
  bf16* Q;
  bf16* AO;
  bf16* A;
  float* attO;
  float2* attML;
  float* ssq;                           // [NORM_PARTS][n_alloc]
  unsigned long long* amax;
  unsigned long long* sec;              // [tiles][n_alloc] second-best packed key of every vocabulary tile, or null
  float2* lse;                          // [tiles][n_alloc] (max, sum of exp(x - max)) of every vocabulary tile, or null
  float* logits;
  const int32_t* pos;
  const unsigned long long* anc;
#ifdef SPECASR_TRACE
  TraceBuf tr;
#endif
};

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int32_t* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_release_add(int32_t* p, int v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// generic-proxy accesses (ordinary loads / stores) <-> async-proxy accesses (TMA) of the same memory
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
__device__ __forceinline__ void worker_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// One projection as this CTA sees it.
struct Gemm {
  const CUtensorMap* tmW;
  int M, K, KB, Kt, tiles, groups, splits;   // tiles of 128 rows in groups of TM; splits > 0: linear output in `splits` k-parts per group
  int g_eff;                            // CTAs that take part
  int U, u0, u1;                        // all (tile group, k-block) units; this CTA's range
};

__device__ __forceinline__ Gemm gemm_of(const StackParams& p, int layer, int which, int cta, int G) {
  Gemm g;
  switch (which) {
    case ST_QKV: g.M = p.qkv_dim; g.K = p.d; g.splits = p.splits_qkv; g.tmW = p.w_maps + 4 * layer; break;
    case ST_O: g.M = p.d; g.K = p.q_dim; g.splits = p.splits_o; g.tmW = p.w_maps + 4 * layer + 1; break;
    case ST_GU: g.M = 2 * p.ffn; g.K = p.d; g.splits = 0; g.tmW = p.w_maps + 4 * layer + 2; break;
    case ST_DOWN: g.M = p.d; g.K = p.ffn; g.splits = p.splits_down; g.tmW = p.w_maps + 4 * layer + 3; break;
    default: g.M = p.vocab; g.K = p.d; g.splits = 0; g.tmW = p.w_maps + 4 * p.n_layers; break;      // vocabulary
  }
  g.KB = (g.K + KSUB * SUB_K - 1) / (KSUB * SUB_K);
  g.Kt = packed_col_tiles(g.K);
  g.tiles = (g.M + TILE_M - 1) / TILE_M;
  g.groups = (g.tiles + TM - 1) / TM;
  g.U = g.groups * g.KB;
  if (g.splits > 0) {
    g.g_eff = g.groups * g.splits;
    if (cta < g.g_eff) {
      const int tile = cta / g.splits, split = cta % g.splits;
      g.u0 = tile * g.KB + split * g.KB / g.splits;
      g.u1 = tile * g.KB + (split + 1) * g.KB / g.splits;
    } else {
      g.u0 = g.u1 = 0;
    }
  } else {
    g.g_eff = g.U < G ? g.U : G;
    if (cta < g.g_eff) {
      g.u0 = (int)((long long)cta * g.U / g.g_eff);
      g.u1 = (int)((long long)(cta + 1) * g.U / g.g_eff);
    } else {
      g.u0 = g.u1 = 0;
    }
  }
  return g;
}

// The projection that step `st` of layer `l` runs (l == n_layers: final norm at st 0, vocabulary projection at st 1),
// or -2 if the step is not a projection.  Every role walks the steps in one loop, so that each piece of code has a
// single call site: the kernel's instructions are fetched again on every layer, and their size is time.
__device__ __forceinline__ int gemm_kind_of(int l, int st, int n_layers) {
  if (l == n_layers) return st == 1 ? -1 : -2;
  return (st == ST_QKV || st == ST_O || st == ST_GU || st == ST_DOWN) ? st : -2;
}

// The polling loops are kept out of line: the kernel has some forty waits, and its text is fetched again on every
// layer, so a copy of the loop at each of them is paid for in instruction-cache misses.
__device__ __noinline__ bool bar_wait(void* bar, uint32_t parity, volatile int* abort, int32_t* status) {
  return mbar_wait(bar, parity, abort, status);
}
__device__ __noinline__ bool bar_wait_relaxed(void* bar, uint32_t parity, volatile int* abort, int32_t* status) {
  return mbar_wait_relaxed(bar, parity, abort, status);
}

// Bounded poll of a word that only grows.  Returns false when the limit ran out or the call was aborted.
__device__ __noinline__ bool wait_word_ge(const int32_t* word, int target, volatile int* abort, int32_t* status) {
  if (ld_acquire(word) >= target) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    __nanosleep(20);
    if (ld_acquire(word) >= target) return true;
    if ((it & 15u) == 0u) {
      if (*abort) return false;
      if (*(volatile int32_t*)status != 0) {
        *abort = 1;
        return false;
      }
      if (global_ns() - t0 > WAIT_LIMIT_NS) {
        *abort = 1;
        atomicExch(status, (int32_t)SPECASR_ERR_TIMEOUT);
        return false;
      }
    }
  }
}
__device__ __noinline__ bool wait_smem_ge(volatile int* word, int target, volatile int* abort, int32_t* status) {
  if (*word >= target) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    __nanosleep(40);
    if (*word >= target) return true;
    if ((it & 15u) == 0u) {
      if (*abort) return false;
      if (global_ns() - t0 > WAIT_LIMIT_NS) {
        *abort = 1;
        atomicExch(status, (int32_t)SPECASR_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

// The utterance that owns workspace row `row` (segments are laid out back to back in table order).
__device__ __forceinline__ int seg_of_row(const SegTable& tab, int row) {
  int b = 0;
  while (b + 1 < tab.count && row >= tab.seg[b].row0 + tab.seg[b].n) ++b;
  return b;
}

// Device-side trace (build variant): worker thread 0 of every CTA appends one record per step
// {kind | (layer + 1) << 8, start, end, time its wait for the previous steps ended} and, at a few points inside a
// step, point records {(100 + point) | (layer + 1) << 8, now, now, 0}.
#ifdef SPECASR_TRACE
#define STACK_TRACE_BEGIN() unsigned long long tr_t0_ = wtid == 0 ? global_ns() : 0ull, tr_mark_ = tr_t0_
#define STACK_TRACE_MARK() do { if (wtid == 0) tr_mark_ = global_ns(); } while (0)
#define STACK_TRACE_WRITE(code, layer, a, b, c)                                          \
  do {                                                                                   \
    if (wtid == 0 && p.tr.buf != nullptr) {                                              \
      const unsigned long long slot_ = atomicAdd(p.tr.buf, 1ull);                        \
      if (slot_ < p.tr.cap) {                                                            \
        unsigned long long* e_ = p.tr.buf + 2 + slot_ * 4;                               \
        e_[0] = (unsigned long long)(code) | ((unsigned long long)((layer) + 1) << 8);   \
        e_[1] = (a);                                                                     \
        e_[2] = (b);                                                                     \
        e_[3] = (c);                                                                     \
      }                                                                                  \
    }                                                                                    \
  } while (0)
#define STACK_TRACE_END(kind, layer) STACK_TRACE_WRITE(kind, layer, tr_t0_, global_ns(), tr_mark_)
#define STACK_TRACE_POINT(point, layer)                                                  \
  do {                                                                                   \
    if (wtid == 0 && p.tr.buf != nullptr && p.tr.buf[1] != 0ull) {   /* word 1 of the buffer switches points on */                               \
      const unsigned long long now_ = global_ns();                                       \
      STACK_TRACE_WRITE(100 + (point), layer, now_, now_, (unsigned long long)blockIdx.x);                         \
    }                                                                                    \
  } while (0)
#else
#define STACK_TRACE_BEGIN()
#define STACK_TRACE_MARK()
#define STACK_TRACE_END(kind, layer)
#define STACK_TRACE_POINT(point, layer)
#endif

template <int DH>
__global__ void __launch_bounds__(NUM_THREADS, 1)
k_stack(const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmAO,
        const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmQ,
        const __grid_constant__ SegTable tab, const StackParams p) {
  constexpr int H2 = DH / 64;                           // 64-wide halves of a head
  constexpr int A_BYTES = 4 * SUB;                      // Q planes, later two P planes of 128 keys
  extern __shared__ uint8_t smem_raw[];
  uint8_t* ring = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  StackCtl* sc = (StackCtl*)(ring + p.ring_bytes);
  bf16* epi_stage = (bf16*)(sc + 1);                    // SiLU * up output tile [2 planes][tokens][64]
  uint8_t* As = ring;                                   // attention: overlays the ring
  uint8_t* KVs = ring + A_BYTES;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = gridDim.x, cta = blockIdx.x;
  const int n_pad = p.n_pad;
  const int act_sub = n_pad * 2 * SUB_K * 2;            // both planes of one 64-wide k sub-block
  const int act_stage = KSUB * act_sub;
  const int acc_cols = 2 * n_pad;                       // hi | lo halves of one accumulator set

  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_STAGES; ++s) {
      mbar_init(&sc->full[s], 2);                       // weight producer + activation producer
      mbar_init(&sc->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sc->acc_full[b], 1);
      mbar_init(&sc->acc_empty[b], WORKERS);
      mbar_init(&sc->bar_p[b], WORKERS);
      mbar_init(&sc->bar_o[b], 1);
    }
    mbar_init(&sc->bar_qk, 1);
    mbar_init(&sc->bar_v, 1);
    mbar_init(&sc->bar_s, 1);
    sc->abort = 0;
    sc->attn_done = 0;
    sc->units_done = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmH);
    tma_prefetch_desc(&tmAO);
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmQ);
  }
  if (warp == 1) tmem_alloc(&sc->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sc->tmem_base;
  volatile int* abort = &sc->abort;
  int32_t* status = p.ctl + CTL_STATUS;
  const bool live = *(volatile int32_t*)status == 0;
  const int n_steps = p.n_layers * ST_PER_LAYER + (p.want_head ? 2 : 0);   // final norm and vocabulary projection last

  // attention geometry shared by all roles
  const int rows_used = p.nodes_per_tile * p.group;

  if (!live) {
    // the call was refused before it started (shared status): nothing to do
  } else if (warp == 0 && lane == 0) {
    // =========================================================== weight producer
    // A cursor walks this CTA's (layer, projection, unit) list, which is fixed for the call, and issues the TMA loads
    // into the ring as slots come free: weights never wait for a step, so the first tiles of the next projection
    // are in shared memory before its input exists.  (Asking for units further ahead to be brought into L2 --
    // continuously, or only while the attention step holds the ring -- measured slower at every depth tried.)
    struct Cursor {
      int l, ph;                 // layer; 0..3 = QKV, O, gate/up, down; layer == n_layers: the vocabulary projection
      int u, u1, tile, kb, KB;   // next unit, end of the range, and the unit as (weight tile group, k-block)
      int Kt, tiles;             // 64-wide column tiles per row tile of the packed matrix; its row tiles
      const CUtensorMap* tmW;
      bool done;
    };
    auto phase_of = [&](int ph) { return ph == 0 ? ST_QKV : ph == 1 ? ST_O : ph == 2 ? ST_GU : ST_DOWN; };
    auto settle = [&](Cursor& c) {                       // enter the next phase that has a unit for this CTA
      while (!c.done && c.u >= c.u1) {
        if (c.l >= p.n_layers) {
          c.done = true;
          break;
        }
        if (++c.ph == 4) {
          c.ph = 0;
          ++c.l;
        }
        Gemm g;
        if (c.l < p.n_layers) g = gemm_of(p, c.l, phase_of(c.ph), cta, G);
        else if (p.want_head) g = gemm_of(p, 0, -1, cta, G);
        else {
          c.done = true;
          break;
        }
        c.u = g.u0; c.u1 = g.u1; c.KB = g.KB; c.tmW = g.tmW; c.Kt = g.Kt; c.tiles = g.tiles;
        c.tile = g.u0 / g.KB;
        c.kb = g.u0 % g.KB;
      }
    };
    auto advance = [&](Cursor& c) {
      ++c.u;
      if (++c.kb == c.KB) {
        c.kb = 0;
        ++c.tile;
      }
      if (c.u >= c.u1) settle(c);
    };
    Cursor ld;
    ld.l = 0; ld.ph = -1; ld.u = ld.u1 = 0; ld.tile = ld.kb = 0; ld.KB = 1; ld.Kt = 2; ld.tiles = 1; ld.tmW = nullptr; ld.done = false;
    settle(ld);
    int slot = 0;                                        // next ring slot
    uint32_t ring_par = 0u;                              // parity of the ring round in progress
    int attn_waited = 0;                                 // attention steps whose end this thread has seen
    bool ok = true;
    while (!ld.done && ok) {
      // the attention step of layer l owns the ring between that layer's QKV and O projections
      const int need = ld.l < p.n_layers ? (ld.ph == 0 ? ld.l : ld.l + 1) : p.n_layers;
      if (need > attn_waited) {
        ok = wait_smem_ge(&sc->attn_done, need, abort, status);
        attn_waited = need;
        if (!ok) break;
      }
      if (!bar_wait(&sc->empty[slot], ring_par ^ 1u, abort, status)) {
        ok = false;
        break;
      }
      uint8_t* st = ring + (size_t)slot * p.stage_bytes;
      mbar_expect_tx(&sc->full[slot], (uint32_t)W_STAGE_BYTES);
      for (int t = 0; t < TM; ++t) {                     // tile-packed weights: 16 KB contiguous per box, padding is zeros
        // a group past the last row tile reads that tile again (its accumulator is never looked at)
        const int tile = min(ld.tile * TM + t, ld.tiles - 1);
        for (int q = 0; q < KSUB; ++q)
          tma_load_2d(st + (t * KSUB + q) * W_SUB_BYTES, ld.tmW, 0, (tile * ld.Kt + ld.kb * KSUB + q) * TILE_M,
                      &sc->full[slot]);
      }
      advance(ld);
      if (++slot == p.stages) {
        slot = 0;
        ring_par ^= 1u;
      }
    }
  } else if (warp == 10) {
    // =========================================================== activation producer / attention producer
    int it = 0;
    bool ok = true;
    int au = 0;                                          // attention units this CTA has run
    auto stream_acts = [&](const Gemm& g, const CUtensorMap* tmAct, int ready_step) {
      if (g.u1 <= g.u0) return;
      if (lane == 0) {
        ok = wait_word_ge(p.sync + ready_step, G, abort, status);
        fence_proxy_async_all();
        int kb = g.u0 % g.KB;
        for (int u = g.u0; u < g.u1 && ok; ++u, ++it) {
          const int s = it % p.stages;
          if (!bar_wait(&sc->empty[s], (uint32_t)((it / p.stages) & 1) ^ 1u, abort, status)) {
            ok = false;
            break;
          }
          uint8_t* st = ring + (size_t)s * p.stage_bytes + W_STAGE_BYTES;
          mbar_expect_tx(&sc->full[s], (uint32_t)act_stage);
          for (int q = 0; q < KSUB; ++q)
            tma_load_3d(st + q * act_sub, tmAct, (kb * KSUB + q) * SUB_K, 0, 0, &sc->full[s]);
          if (++kb == g.KB) kb = 0;
        }
      }
      ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
      it = __shfl_sync(0xFFFFFFFFu, it, 0);
    };
    for (int sidx = 0; sidx < n_steps && ok; ++sidx) {
      const int l = sidx / ST_PER_LAYER, st = sidx - l * ST_PER_LAYER;
      const int gk = gemm_kind_of(l, st, p.n_layers);
      if (gk != -2) {
        // the step before a projection is the one that writes its input
        const CUtensorMap* tmAct = gk == ST_O ? &tmAO : gk == ST_DOWN ? &tmA : &tmH;
        stream_acts(gemm_of(p, l, gk, cta, G), tmAct, sidx - 1);
      } else if (l < p.n_layers && st == ST_ATTN) {
        // ---- attention units of this CTA: lane 0 fetches Q, lane j page j of K and later of V.
        // (Asking for the K pages of a key block inside the committed prefix before the rotary step has finished
        // made S ready 1.6 us earlier and the step no shorter; it was taken out again.)
        bool rope_seen = false;
        for (int u = cta; u < p.attn_units && ok; u += G) {
          const int kvh = u % p.Hkv, tile_y = (u / p.Hkv) % p.row_tiles, z = u / (p.Hkv * p.row_tiles);
          const int split = z % tab.splits;
          const SegDev& sg = tab.seg[z / tab.splits];
          const int node0 = tile_y * p.nodes_per_tile;
          if (node0 >= sg.n || sg.ctl[CTL_STATUS] != 0) continue;
          const int L = sg.ctl[CTL_LEN];
          const int Ltot = L + sg.n;
          const int k_begin = split * sg.chunk;
          if (k_begin >= Ltot) continue;
          const int kc = min(sg.chunk, Ltot - k_begin);
          const int pages = (kc + p.page_size - 1) / p.page_size;
          const uint32_t par = (uint32_t)(au & 1);
          ++au;
          auto wait_rope = [&]() {
            if (lane == 0) {
              ok = wait_word_ge(p.sync + sidx - 1, G, abort, status);
              fence_proxy_async_all();
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            rope_seen = true;
          };
          if (!rope_seen) wait_rope();
          // A CTA that runs several units reuses the Q / P and K / V tiles and the barriers: the next unit's loads
          // (and the arming of its barriers) wait until the workers have stored the previous unit's output.
          if (ok && lane == 0) ok = wait_smem_ge(&sc->units_done, au - 1, abort, status);
          ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
          if (!ok) break;
          int my_page = 0;
          if (lane < pages) my_page = sg.page_table[split * (sg.chunk / p.page_size) + lane];
          const uint32_t q_bytes = 2 * H2 * rows_used * 128;
          const uint32_t kv_bytes = 2 * H2 * pages * p.page_size * 128;
          if (lane == 0) {
            mbar_expect_tx(&sc->bar_qk, q_bytes + kv_bytes);
            mbar_expect_tx(&sc->bar_v, kv_bytes);
          }
          __syncwarp();
          const int c4 = l * sg.n_pages + my_page;
          const int off = lane * p.page_size * 128;
          if (lane < pages) {
            for (int plane = 0; plane < 2; ++plane)
              for (int h = 0; h < H2; ++h)
                tma_load_5d(KVs + (plane * H2 + h) * KVSUB + off, sg.tmK, h * 64, 0, plane, kvh, c4, &sc->bar_qk);
          }
          if (lane == 0) {
            for (int plane = 0; plane < 2; ++plane)
              for (int h = 0; h < H2; ++h)
                tma_load_4d(As + (plane * H2 + h) * SUB, &tmQ, h * 64, kvh * p.group, sg.row0 + node0, plane, &sc->bar_qk);
          }
          // V takes K's place once the S MMAs have read K
          ok = bar_wait(&sc->bar_s, par, abort, status);
          if (ok && lane < pages) {
            for (int plane = 0; plane < 2; ++plane)
              for (int h = 0; h < H2; ++h)
                tma_load_5d(KVs + (plane * H2 + h) * KVSUB + off, sg.tmV, h * 64, 0, plane, kvh, c4, &sc->bar_v);
          }
          ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
        }
      }
    }
  } else if (warp == 1 && lane == 0) {
    // =========================================================== MMA issuer
    int it = 0, seg = 0, au = 0, au2 = 0;
    bool ok = true;
    const uint32_t idesc = make_idesc_bf16(2 * n_pad);
    auto run_gemm = [&](const Gemm& g) {
      for (int u = g.u0; u < g.u1 && ok; ++seg) {
        const int kb0 = u % g.KB;
        const int kb1 = (g.u1 - u) < (g.KB - kb0) ? kb0 + (g.u1 - u) : g.KB;
        const int b = seg & 1;
        if (!bar_wait(&sc->acc_empty[b], (uint32_t)((seg >> 1) & 1) ^ 1u, abort, status)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t d_addr = tmem_base + (uint32_t)(b * TM * acc_cols);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % p.stages;
          if (!bar_wait(&sc->full[s], (uint32_t)((it / p.stages) & 1), abort, status)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t w_lo = smem_desc_lo(smem_u32(ring + (size_t)s * p.stage_bytes));
          const uint32_t act_lo = w_lo + (W_STAGE_BYTES >> 4);
#pragma unroll
          for (int t = 0; t < TM; ++t) {
#pragma unroll
            for (int q = 0; q < KSUB; ++q) {
#pragma unroll
              for (int k = 0; k < SUB_K / UMMA_K; ++k) {
                const uint32_t acc = (q > 0 || k > 0) ? 1u : (kb > kb0 ? 1u : 0u);
                umma_bf16_lo(d_addr + (uint32_t)(t * acc_cols), w_lo + (((t * KSUB + q) * W_SUB_BYTES + k * UMMA_K * 2) >> 4),
                             act_lo + ((q * act_sub + k * UMMA_K * 2) >> 4), idesc, acc);
              }
            }
          }
          umma_commit(&sc->empty[s]);                    // arrives once these MMAs have read the stage
        }
        if (ok) umma_commit(&sc->acc_full[b]);
        u += kb1 - kb0;
      }
    };
    for (int sidx = 0; sidx < n_steps && ok; ++sidx) {
      const int l = sidx / ST_PER_LAYER, st = sidx - l * ST_PER_LAYER;
      const int gk = gemm_kind_of(l, st, p.n_layers);
      if (gk != -2) {
        run_gemm(gemm_of(p, l, gk, cta, G));
      } else if (l < p.n_layers && st == ST_ATTN) {
        // ---- attention units
        for (int u = cta; u < p.attn_units && ok; u += G) {
          const int tile_y = (u / p.Hkv) % p.row_tiles, z = u / (p.Hkv * p.row_tiles);
          const int split = z % tab.splits;
          const SegDev& sg = tab.seg[z / tab.splits];
          if (tile_y * p.nodes_per_tile >= sg.n || sg.ctl[CTL_STATUS] != 0) continue;
          const int Ltot = sg.ctl[CTL_LEN] + sg.n;
          const int k_begin = split * sg.chunk;
          if (k_begin >= Ltot) continue;
          const int kc = min(sg.chunk, Ltot - k_begin);
          const int kc_pad = (kc + 15) & ~15;
          const int rounds = (kc_pad + ROUND - 1) / ROUND;
          const uint32_t par = (uint32_t)(au & 1);
          ++au;
          const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + 256;
          ok = bar_wait(&sc->bar_qk, par, abort, status);
          if (!ok) break;
          tc_fence_after();
          {
            const uint32_t idesc_s = make_idesc_bf16(kc_pad);
            const uint32_t a_lo = smem_desc_lo(smem_u32(As)), b_lo = smem_desc_lo(smem_u32(KVs));
  #pragma unroll
            for (int term = 0; term < 3; ++term) {       // straight-line: a few instructions per MMA
              const int qp = term == 2 ? 1 : 0, kp = term == 1 ? 1 : 0;     // hi*hi, hi*lo, lo*hi
  #pragma unroll
              for (int h = 0; h < H2; ++h) {
  #pragma unroll
                for (int k = 0; k < 4; ++k)
                  umma_bf16_lo(tmem_s, a_lo + (((qp * H2 + h) * SUB + k * 32) >> 4),
                               b_lo + (((kp * H2 + h) * KVSUB + k * 32) >> 4), idesc_s, (term | h | k) ? 1u : 0u);
              }
            }
            umma_commit(&sc->bar_s);
          }
          ok = bar_wait(&sc->bar_v, par, abort, status);
          const uint32_t idesc2 = make_idesc_bf16(DH, true);
          uint32_t acc = 0u;
          for (int rd = 0; rd < rounds && ok; ++rd) {
            const uint32_t par_r = rd == 0 ? par : (uint32_t)(au2 & 1);
            ok = bar_wait(&sc->bar_p[rd], par_r, abort, status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_lo = smem_desc_lo(smem_u32(As));
            const uint32_t b_lo = smem_desc_lo(smem_u32(KVs), KVSUB) + (uint32_t)((rd * (ROUND / 16) * 2048) >> 4);
            const int j_end = min(kc_pad - rd * ROUND, ROUND) / 16;
  #pragma unroll
            for (int term = 0; term < 3; ++term) {
              const int pp = term == 2 ? 1 : 0, vp = term == 1 ? 1 : 0;
  #pragma unroll
              for (int j = 0; j < ROUND / 16; ++j) {
                if (j < j_end) {
                  umma_bf16_lo(tmem_o, a_lo + (((pp * 2 + (j >> 2)) * SUB + (j & 3) * 32) >> 4),
                               b_lo + ((vp * H2 * KVSUB + j * 2048) >> 4), idesc2, acc);
                  acc = 1u;
                }
              }
            }
            umma_commit(&sc->bar_o[rd]);
          }
          if (rounds == 2) ++au2;
        }
      }
    }
  } else if (warp >= 2 && warp < 10) {
    // =========================================================== workers
    const int wtid = threadIdx.x - 64;
    const int wwarp = warp - 2;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;                   // TMEM lane = output row of a weight tile / query row
    const int c_first = (wwarp >> 2) * 16;              // projections: this warp's first 16-token block, stride 32
    const int eg = wwarp >> 2;                          // attention: which 32-key chunks this thread takes
    const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
    bool ok = true;
    int seg = 0, au = 0, au2 = 0;
    int arrived = 0;                                     // steps this CTA has signed off
    int cur_layer = 0;
    (void)cur_layer;

    // Barriers among the workers (worker_bar) are never placed under a condition that a failed wait could make
    // differ between threads; `ok` only guards waits and memory traffic.  A wait's verdict is made uniform
    // across the warp because the TMEM loads that follow are warp-wide instructions.
    auto wwait = [&](void* bar, uint32_t parity) -> bool {
      return __all_sync(0xFFFFFFFFu, bar_wait(bar, parity, abort, status) ? 1 : 0) != 0;
    };
    auto wwait_relaxed = [&](void* bar, uint32_t parity) -> bool {
      return __all_sync(0xFFFFFFFFu, bar_wait_relaxed(bar, parity, abort, status) ? 1 : 0) != 0;
    };
    // every worker's global writes of the step are done and visible -> one arrival for the CTA
    auto arrive_step = [&]() {
      worker_bar();                                      // every worker's stores of the step are issued ...
      if (wtid == 0) {
        __threadfence();                                 // ... and ordered before the arrival (cumulative over the barrier)
        fence_proxy_async_global();                      // the next step may read them through TMA
        red_release_add(p.sync + arrived, 1);
      }
      ++arrived;
    };
    // all CTAs have signed off step `step`
    auto wait_step = [&](int step) {
      if (wtid == 0) sc->step_ok = (ok && wait_word_ge(p.sync + step, G, abort, status)) ? 1 : 0;
      worker_bar();
      ok = ok && sc->step_ok != 0;                       // the same verdict for every worker
    };
    auto worker_sum = [&](float v) -> float {            // fixed order: deterministic
      v = warp_sum(v);
      if (lane == 0) sc->red[wwarp] = v;
      worker_bar();
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) t += sc->red[w];
      worker_bar();
      return t;
    };
    // 1 / rms of every row from the sums of squares the last norm step left
    auto load_inv = [&]() {
      if (wtid < n_pad) {
        float ss = 0.f;
        if (wtid < p.n) {
#pragma unroll
          for (int q = 0; q < NORM_PARTS; ++q) ss += __ldcg(p.ssq + q * p.n_alloc + wtid);
        }
        sc->inv[wtid] = rsqrtf(ss / (float)p.d + p.eps);
      }
      worker_bar();
    };

    // ---------------- norm step: x += planes, h = x * g as hi / lo planes, sums of squares per half row
    auto norm_step = [&](const float* __restrict__ gain, int n_planes, size_t plane_stride) {
      const int d = p.d;
      const int d_part = ((d + NORM_PARTS - 1) / NORM_PARTS + 3) & ~3;
      const int items = p.n * NORM_PARTS;
      const size_t h_plane = (size_t)p.n_alloc * d;
#pragma unroll 1
      for (int item = cta; item < items; item += G) {
        const int r = item / NORM_PARTS, part = item % NORM_PARTS;
        const int k_end = min(d, (part + 1) * d_part);
        float* x = p.X + (size_t)r * d;
        float ss = 0.f;
#pragma unroll 1
        for (int k0 = part * d_part + wtid * 4; k0 < k_end; k0 += 2 * WORKERS * 4) {
          const int k1 = k0 + WORKERS * 4;
          const bool on1 = k1 < k_end;
          float4 v0 = *reinterpret_cast<const float4*>(x + k0);
          float4 v1 = on1 ? *reinterpret_cast<const float4*>(x + k1) : make_float4(0.f, 0.f, 0.f, 0.f);
          const float4 g0 = *reinterpret_cast<const float4*>(gain + k0);
          const float4 g1 = on1 ? *reinterpret_cast<const float4*>(gain + k1) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
          for (int s0 = 0; s0 < n_planes; s0 += 4) {
            float4 q0[4], q1[4];
#pragma unroll
            for (int s = 0; s < 4; ++s) {
              const bool on = s0 + s < n_planes;
              const float* src = p.P + (size_t)(s0 + s) * plane_stride + (size_t)r * d;
              q0[s] = on ? __ldcg(reinterpret_cast<const float4*>(src + k0)) : make_float4(0.f, 0.f, 0.f, 0.f);
              q1[s] = (on && on1) ? __ldcg(reinterpret_cast<const float4*>(src + k1)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int s = 0; s < 4; ++s) {
              v0.x += q0[s].x; v0.y += q0[s].y; v0.z += q0[s].z; v0.w += q0[s].w;
              v1.x += q1[s].x; v1.y += q1[s].y; v1.z += q1[s].z; v1.w += q1[s].w;
            }
          }
          if (n_planes > 0) {
            *reinterpret_cast<float4*>(x + k0) = v0;
            if (on1) *reinterpret_cast<float4*>(x + k1) = v1;
          }
          ss += v0.x * v0.x + v0.y * v0.y + v0.z * v0.z + v0.w * v0.w;
          ss += v1.x * v1.x + v1.y * v1.y + v1.z * v1.z + v1.w * v1.w;
          bf16* hi = p.H + (size_t)r * d;
          uint32_t ph[2], pl[2];
          split2_pack(v0.x * g0.x, v0.y * g0.y, ph[0], pl[0]);
          split2_pack(v0.z * g0.z, v0.w * g0.w, ph[1], pl[1]);
          *reinterpret_cast<uint2*>(hi + k0) = make_uint2(ph[0], ph[1]);
          *reinterpret_cast<uint2*>(hi + h_plane + k0) = make_uint2(pl[0], pl[1]);
          if (on1) {
            split2_pack(v1.x * g1.x, v1.y * g1.y, ph[0], pl[0]);
            split2_pack(v1.z * g1.z, v1.w * g1.w, ph[1], pl[1]);
            *reinterpret_cast<uint2*>(hi + k1) = make_uint2(ph[0], ph[1]);
            *reinterpret_cast<uint2*>(hi + h_plane + k1) = make_uint2(pl[0], pl[1]);
          }
        }
        ss = worker_sum(ss);
        if (wtid == 0) p.ssq[part * p.n_alloc + r] = ss;
      }
    };

    // ---------------- projection epilogues
    auto load16 = [&](uint32_t lane_addr, int c0, float* v) {     // hi half + lo half of the accumulator
      float lo[16];
      tmem_ld16x2(lane_addr + (uint32_t)c0, lane_addr + (uint32_t)(c0 + n_pad), v, lo);
#pragma unroll
      for (int j = 0; j < 16; ++j) v[j] += lo[j];
    };
    // linear output: fp32 partial plane `split`
    auto epi_partial = [&](const Gemm& g, size_t plane_stride) {
#pragma unroll 1
      for (int u = g.u0; u < g.u1; ++seg) {
        const int grp = u / g.KB;
        const int kb0 = u % g.KB;
        const int kb1 = (g.u1 - u) < (g.KB - kb0) ? kb0 + (g.u1 - u) : g.KB;
        u += kb1 - kb0;
        const int b = seg & 1;
        if (ok) ok = wwait_relaxed(&sc->acc_full[b], (uint32_t)((seg >> 1) & 1));
        STACK_TRACE_POINT(10, cur_layer);
        tc_fence_after();
        if (!ok) continue;
        float* out = p.P + (size_t)(cta % g.splits) * plane_stride;
#pragma unroll 1
        for (int t = 0; t < TM; ++t) {
          const uint32_t lane_addr = tmem_base + lane_off + (uint32_t)((b * TM + t) * acc_cols);
          const int m = (grp * TM + t) * TILE_M + row;
#pragma unroll 1
          for (int c0 = c_first; c0 < n_pad; c0 += 32) {
            float v[16];
            load16(lane_addr, c0, v);
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (c0 + j < p.n && m < g.M) out[(size_t)(c0 + j) * g.M + m] = v[j];
          }
        }
        tc_fence_before();
        mbar_arrive(&sc->acc_empty[b]);
      }
    };
    // SiLU(gate) * up (swiglu = true) or arg-max over the vocabulary (swiglu = false), equal unit ranges
    auto epi_streamk = [&](const Gemm& g, bool swiglu, int epoch) {
#pragma unroll 1
      for (int u = g.u0; u < g.u1; ++seg) {
        const int grp = u / g.KB;
        const int kb0 = u % g.KB;
        const int kb1 = (g.u1 - u) < (g.KB - kb0) ? kb0 + (g.u1 - u) : g.KB;
        u += kb1 - kb0;
        const int b = seg & 1;
        // the CTA that holds the first k-blocks of a split tile group adds what the CTAs holding the rest have parked
        int last = cta;
        if (kb0 == 0 && kb1 != g.KB)
          while (last + 1 < g.g_eff && (long long)(last + 1) * g.U / g.g_eff < (long long)(grp + 1) * g.KB) ++last;
        float pk0[16], pk1[16];
        auto load_parked = [&](int t, int c0, float* f) {
#pragma unroll
          for (int j = 0; j < 16; ++j) f[j] = 0.f;
          if (c0 < n_pad)
#pragma unroll 1
            for (int cc = cta + 1; cc <= last; ++cc) {
              const float* src = p.fixP + (((size_t)cc * TM + t) * n_pad + c0) * TILE_M + row;
#pragma unroll
              for (int j = 0; j < 16; ++j) f[j] += __ldcg(src + j * TILE_M);
            }
        };
        if (last > cta) {
          if (wtid == 0) {
            bool got = ok;
#pragma unroll 1
            for (int cc = cta + 1; cc <= last && got; ++cc)
              got = wait_word_ge(p.fixFlag + cc, epoch, abort, status);            // flags carry the launch's epoch
            sc->step_ok = got ? 1 : 0;
          }
          worker_bar();
          ok = ok && sc->step_ok != 0;
        }
        if (ok) ok = wwait_relaxed(&sc->acc_full[b], (uint32_t)((seg >> 1) & 1));
        STACK_TRACE_POINT(kb0 != 0 ? 12 : 11, cur_layer);
        tc_fence_after();
        const uint32_t lane_base = tmem_base + lane_off + (uint32_t)(b * TM * acc_cols);

        if (kb0 != 0) {
          // later k-blocks of a group whose first k-blocks belong to an earlier CTA: park the partial sums
          float* dst = p.fixP + (size_t)cta * TM * n_pad * TILE_M;
          if (ok) {
#pragma unroll 1
            for (int t = 0; t < TM; ++t) {
              if ((grp * TM + t) >= g.tiles) break;
#pragma unroll 1
              for (int c0 = c_first; c0 < n_pad; c0 += 32) {
                float v[16];
                load16(lane_base + (uint32_t)(t * acc_cols), c0, v);
#pragma unroll
                for (int j = 0; j < 16; ++j) dst[((size_t)t * n_pad + c0 + j) * TILE_M + row] = v[j];
              }
            }
            tc_fence_before();
            mbar_arrive(&sc->acc_empty[b]);
            __threadfence();
          }
          worker_bar();
          if (ok && wtid == 0) st_release(p.fixFlag + cta, epoch);
          continue;
        }

#pragma unroll 1
        for (int t = 0; t < TM; ++t) {
        const int tile = grp * TM + t;
        if (tile >= g.tiles) break;
        const uint32_t lane_addr = lane_base + (uint32_t)(t * acc_cols);
        if (last > cta && ok) {
          load_parked(t, c_first, pk0);
          load_parked(t, c_first + 32, pk1);
        }
        const int m = tile * TILE_M + row;
        const bool row_ok = m < g.M;
        if (!swiglu) {
          if (wtid < 64) sc->key[wtid] = 0ull;
          worker_bar();
        }
        if (ok) {
#pragma unroll 1
          for (int c0 = c_first; c0 < n_pad; c0 += 32) {
            float v[16];
            load16(lane_addr, c0, v);
            if (last > cta) {
              const bool first = c0 == c_first;
#pragma unroll
              for (int j = 0; j < 16; ++j) v[j] += first ? pk0[j] : pk1[j];
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] *= sc->inv[c0 + j];
            if (swiglu) {
              // rows 2f / 2f + 1 of the tile are gate / up of feature f: the even lane keeps the hi plane of the
              // product, the odd lane the lo plane, staged in shared memory for 16-byte global stores
              float a[16];
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                const float other = __shfl_xor_sync(0xFFFFFFFFu, v[j], 1);
                const float gt = (lane & 1) ? other : v[j];
                const float up = (lane & 1) ? v[j] : other;
                a[j] = __fdividef(gt, 1.f + __expf(-gt)) * up;
              }
              bf16* st = epi_stage + (size_t)(lane & 1) * n_pad * 64 + (size_t)c0 * 64 + (row >> 1);
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                bf16 hi, lo;
                split_bf16(a[j], hi, lo);
                st[j * 64] = (lane & 1) ? lo : hi;
              }
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                const int t = c0 + j;
                if (p.logits && t < p.n && row_ok) p.logits[(size_t)t * g.M + m] = v[j];
                uint32_t key = __float_as_uint(v[j]);
                key = (key & 0x80000000u) ? ~key : (key | 0x80000000u);
                if (!row_ok) key = 0u;
                const uint32_t best = __reduce_max_sync(0xFFFFFFFFu, key);
                const uint32_t who = __reduce_min_sync(0xFFFFFFFFu, key == best ? (uint32_t)m : 0xFFFFFFFFu);
                if (lane == 0 && t < p.n && best != 0u)
                  atomicMax(&sc->key[t], ((unsigned long long)best << 32) | (unsigned long long)(0xFFFFFFFFu - who));
                if (p.sec != nullptr) {
                  // the draft side also wants the runner-up and the softmax denominator (Sections IV-A, IV-C): second
                  // largest key of this warp's 32 rows, and the sum of exp(x - warp max)
                  const uint32_t key2 = (uint32_t)m != who ? key : 0u;
                  const uint32_t sbest = __reduce_max_sync(0xFFFFFFFFu, key2);
                  const uint32_t swho = __reduce_min_sync(0xFFFFFFFFu, key2 == sbest ? (uint32_t)m : 0xFFFFFFFFu);
                  const uint32_t ub = (best & 0x80000000u) ? (best & 0x7FFFFFFFu) : ~best;
                  const float vmax = __uint_as_float(ub);
                  const float esum = warp_sum((row_ok && best != 0u) ? __expf(v[j] - vmax) : 0.f);
                  if (lane == 0 && t < p.n) {
                    sc->k1q[quad][t] = best != 0u ? ((unsigned long long)best << 32) | (unsigned long long)(0xFFFFFFFFu - who) : 0ull;
                    sc->k2q[quad][t] = sbest != 0u ? ((unsigned long long)sbest << 32) | (unsigned long long)(0xFFFFFFFFu - swho) : 0ull;
                    sc->msq[quad][t] = best != 0u ? make_float2(vmax, esum) : make_float2(-INFINITY, 0.f);
                  }
                }
              }
            }
          }
        }
        worker_bar();
        if (ok) {
          if (swiglu) {
            const int F = g.M >> 1;
            const int f0 = tile * 64;
            const int nt = p.n;
            const int chunks = 2 * nt * 8;                    // 16-byte pieces of the [2][nt][64] tile
#pragma unroll 1
            for (int idx = wtid; idx < chunks; idx += WORKERS) {
              const int plane = idx / (nt * 8), rem = idx % (nt * 8);
              const int t = rem >> 3, ch = rem & 7;
              if (f0 + ch * 8 < F)
                *reinterpret_cast<uint4*>(p.A + (size_t)plane * p.n_alloc * F + (size_t)t * F + f0 + ch * 8) =
                    *reinterpret_cast<const uint4*>(epi_stage + (size_t)plane * n_pad * 64 + t * 64 + ch * 8);
            }
          } else {
#pragma unroll 1
            for (int t = wtid; t < p.n; t += WORKERS) {
              p.amax[(size_t)tile * p.n_alloc + t] = sc->key[t];
              if (p.sec != nullptr) {                          // the four quadrants of the tile, in a fixed order
                unsigned long long a = 0ull, b = 0ull;
                float mm = -INFINITY, ss = 0.f;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  const unsigned long long c1 = sc->k1q[q][t], c2 = sc->k2q[q][t];     // c1 > c2, all keys distinct or 0
                  if (c1 > a) {
                    b = a;
                    a = c1;
                  } else if (c1 > b) {
                    b = c1;
                  }
                  if (c2 > b) b = c2;                                                   // c2 < c1 <= a
                  const float2 ms = sc->msq[q][t];
                  const float mx = fmaxf(mm, ms.x);
                  if (mx > -INFINITY) {
                    ss = ss * __expf(mm - mx) + ms.y * __expf(ms.x - mx);
                    mm = mx;
                  }
                }
                p.sec[(size_t)tile * p.n_alloc + t] = b;
                p.lse[(size_t)tile * p.n_alloc + t] = make_float2(mm, ss);
              }
            }
          }
        }
        worker_bar();
        }
        if (ok) {
          tc_fence_before();
          mbar_arrive(&sc->acc_empty[b]);
        }
      }
    };

    // ---------------- rotary embedding at tree positions + cache append (from the QKV partial planes)
    auto rope_step = [&](int layer) {
      const int half = DH >> 1;
      const int per_head = half >> 2;                    // threads per head: four rotation pairs each
      const int heads_all = p.Hq + 2 * p.Hkv;
      const long long total = (long long)p.n * heads_all * per_head;
      const size_t pstride = (size_t)p.n_alloc * p.qkv_dim;
      const size_t q_plane = (size_t)p.n_alloc * p.q_dim;
#pragma unroll 1
      for (long long idx = (long long)cta * WORKERS + wtid; idx < total; idx += (long long)G * WORKERS) {
        const int i = (int)(idx / (heads_all * per_head));
        const int rem = (int)(idx % (heads_all * per_head));
        const int head = rem / per_head, k = (rem % per_head) * 4;
        const SegDev& sg = tab.seg[seg_of_row(tab, i)];
        const size_t col = (size_t)i * p.qkv_dim + (size_t)head * DH;
        const size_t c1 = col + qkv_row_of_feature(k, DH), c2 = col + qkv_row_of_feature(k + half, DH);
        const bool is_v = head >= p.Hq + p.Hkv;
        float4 x1 = make_float4(0.f, 0.f, 0.f, 0.f), x2 = x1;
        float4 cs01 = make_float4(1.f, 0.f, 1.f, 0.f), cs23 = cs01;
        float4 a1[4], a2[4];
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          const bool on = s < p.splits_qkv;
          a1[s] = on ? __ldcg(reinterpret_cast<const float4*>(p.P + s * pstride + c1)) : make_float4(0.f, 0.f, 0.f, 0.f);
          a2[s] = on ? __ldcg(reinterpret_cast<const float4*>(p.P + s * pstride + c2)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        const int seg_status = sg.ctl[CTL_STATUS];
        const int len = sg.ctl[CTL_LEN];
        const float ss = __ldcg(p.ssq + i) + __ldcg(p.ssq + p.n_alloc + i);
        if (!is_v) {
          const int pp = min(max(p.pos[i], 0), p.max_positions - 1);
          const float4* t = reinterpret_cast<const float4*>(p.rope + (size_t)pp * half + k);
          cs01 = t[0];
          cs23 = t[1];
        }
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          x1.x += a1[s].x; x1.y += a1[s].y; x1.z += a1[s].z; x1.w += a1[s].w;
          x2.x += a2[s].x; x2.y += a2[s].y; x2.z += a2[s].z; x2.w += a2[s].w;
        }
#pragma unroll 1
        for (int s0 = 4; s0 < p.splits_qkv; s0 += 4) {
#pragma unroll
          for (int s = 0; s < 4; ++s) {
            const bool on = s0 + s < p.splits_qkv;
            a1[s] = on ? __ldcg(reinterpret_cast<const float4*>(p.P + (s0 + s) * pstride + c1)) : make_float4(0.f, 0.f, 0.f, 0.f);
            a2[s] = on ? __ldcg(reinterpret_cast<const float4*>(p.P + (s0 + s) * pstride + c2)) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int s = 0; s < 4; ++s) {
            x1.x += a1[s].x; x1.y += a1[s].y; x1.z += a1[s].z; x1.w += a1[s].w;
            x2.x += a2[s].x; x2.y += a2[s].y; x2.z += a2[s].z; x2.w += a2[s].w;
          }
        }
        if (seg_status != 0) continue;                   // nothing is written for an utterance whose tree was refused
        const float inv = rsqrtf(ss / (float)p.d + p.eps);
        x1.x *= inv; x1.y *= inv; x1.z *= inv; x1.w *= inv;
        x2.x *= inv; x2.y *= inv; x2.z *= inv; x2.w *= inv;
        const float4 r1 = make_float4(x1.x * cs01.x - x2.x * cs01.y, x1.y * cs01.z - x2.y * cs01.w,
                                      x1.z * cs23.x - x2.z * cs23.y, x1.w * cs23.z - x2.w * cs23.w);
        const float4 r2 = make_float4(x2.x * cs01.x + x1.x * cs01.y, x2.y * cs01.z + x1.y * cs01.w,
                                      x2.z * cs23.x + x1.z * cs23.y, x2.w * cs23.z + x1.w * cs23.w);
        uint32_t h1[2], l1[2], h2[2], l2[2];
        split2_pack(r1.x, r1.y, h1[0], l1[0]);
        split2_pack(r1.z, r1.w, h1[1], l1[1]);
        split2_pack(r2.x, r2.y, h2[0], l2[0]);
        split2_pack(r2.z, r2.w, h2[1], l2[1]);
        bf16* dst;
        size_t plane;
        if (head < p.Hq) {
          dst = p.Q + (size_t)i * p.q_dim + (size_t)head * DH;
          plane = q_plane;
        } else {
          const int kvh = is_v ? head - p.Hq - p.Hkv : head - p.Hq;
          const int slot = len + (i - sg.row0);
          const int page = sg.page_table[slot / p.page_size];
          const int off = slot % p.page_size;
          dst = (is_v ? sg.v_pool : sg.k_pool) +
                kv_plane_offset(layer, sg.n_pages, p.Hkv, p.page_size, DH, page, kvh, 0) + (size_t)off * DH;
          plane = (size_t)p.page_size * DH;
        }
        *reinterpret_cast<uint2*>(dst + k) = make_uint2(h1[0], h1[1]);
        *reinterpret_cast<uint2*>(dst + k + half) = make_uint2(h2[0], h2[1]);
        *reinterpret_cast<uint2*>(dst + plane + k) = make_uint2(l1[0], l1[1]);
        *reinterpret_cast<uint2*>(dst + plane + k + half) = make_uint2(l2[0], l2[1]);
      }
    };

    // ---------------- attention: softmax over one key block, unnormalised partial out
    auto attention_step = [&]() {
      const size_t rows_alloc = (size_t)p.n_alloc * p.Hq;
#pragma unroll 1
      for (int u = cta; u < p.attn_units; u += G) {
        const int kvh = u % p.Hkv, tile_y = (u / p.Hkv) % p.row_tiles, z = u / (p.Hkv * p.row_tiles);
        const int split = z % tab.splits;
        const SegDev& sg = tab.seg[z / tab.splits];
        const int node0 = tile_y * p.nodes_per_tile;
        if (node0 >= sg.n || sg.ctl[CTL_STATUS] != 0) continue;
        const int L = sg.ctl[CTL_LEN];
        const int Ltot = L + sg.n;
        const int k_begin = split * sg.chunk;
        const int node = node0 + row / p.group;
        const bool row_valid = row < rows_used && node < sg.n;
        const size_t out_row = (size_t)split * rows_alloc + (size_t)(sg.row0 + node) * p.Hq + kvh * p.group + row % p.group;
        if (k_begin >= Ltot) {                           // key block beyond the cache: an empty partial
          if (row_valid && eg == 0) p.attML[out_row] = make_float2(-INFINITY, 0.f);
          continue;
        }
        const int kc = min(sg.chunk, Ltot - k_begin);
        const int kc_pad = (kc + 15) & ~15;
        const int rounds = (kc_pad + ROUND - 1) / ROUND;
        const uint32_t par = (uint32_t)(au & 1);
        ++au;
        const uint32_t par2 = (uint32_t)(au2 & 1);
        if (rounds == 2) ++au2;
        const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + 256;
        unsigned long long anc0 = 0ull, anc1 = 0ull, anc2 = 0ull, anc3 = 0ull;
        if (row_valid) {
          const unsigned long long* an = p.anc + (size_t)(sg.row0 + node) * 4;
          anc0 = an[0]; anc1 = an[1]; anc2 = an[2]; anc3 = an[3];
        }
        auto visible_keys = [&](int base) -> uint32_t {
          const int t0 = base - L;                      // tree slot of the chunk's first key
          if (t0 <= -32) return 0xFFFFFFFFu;            // all 32 keys lie in the committed prefix
          const int ts = t0 > 0 ? t0 : 0;
          uint32_t win = 0u;                            // ancestor bits of tree slots ts .. ts + 31
          if (ts < SPECASR_MAX_NODES) {
            const int w = ts >> 6, sh = ts & 63;
            const unsigned long long a = w == 0 ? anc0 : w == 1 ? anc1 : w == 2 ? anc2 : anc3;
            const unsigned long long bq = w == 0 ? anc1 : w == 1 ? anc2 : w == 2 ? anc3 : 0ull;
            win = (uint32_t)(sh ? (a >> sh) | (bq << (64 - sh)) : a);
          }
          return t0 < 0 ? ((1u << (-t0)) - 1u) | (win << (-t0)) : win;
        };
        // bit j = key (k_begin + c0 + j) belongs to this unit's block and is visible to this row (16 keys; c0 < kc)
        auto visible16 = [&](int c0) -> uint32_t {
          const uint32_t mine = kc - c0 >= 16 ? 0xFFFFu : (1u << (kc - c0)) - 1u;
          return mine & visible_keys(k_begin + c0);
        };
        if (ok) ok = wwait(&sc->bar_s, par);
        STACK_TRACE_POINT(1, cur_layer);
        float m_row = -INFINITY;
        if (ok) {
          tc_fence_after();
          float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll 1
          for (int c0 = eg * 16; c0 < kc_pad; c0 += 32) {        // short rolled loops: this code runs once per layer
            float s[16];
            tmem_ld16(tmem_s + lane_off + c0, s);
            const uint32_t vis = c0 < kc ? visible16(c0) : 0u;
#pragma unroll
            for (int j = 0; j < 16; ++j) m4[j & 3] = fmaxf(m4[j & 3], ((vis >> j) & 1u) ? s[j] * p.scale_log2 : -INFINITY);
          }
          m_row = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        }
        sc->red_max[eg][row] = m_row;
        STACK_TRACE_POINT(4, cur_layer);
        worker_bar();
        m_row = fmaxf(sc->red_max[0][row], sc->red_max[1][row]);
        const float m_use = m_row > -INFINITY ? m_row : 0.f;      // a fully masked row gives p = 0 everywhere
        float l2[2] = {0.f, 0.f};
#pragma unroll 1
        for (int rd = 0; rd < rounds && ok; ++rd) {
          // the P tile holds 128 keys: the second round waits until the first round's MMAs have read it
          if (rd > 0) ok = wwait(&sc->bar_o[0], par);
          if (!ok) break;
          STACK_TRACE_POINT(5 + rd, cur_layer);
          const int c_end = min(kc_pad, (rd + 1) * ROUND);
#pragma unroll 1
          for (int c0 = rd * ROUND + eg * 16; c0 < c_end; c0 += 32) {
            float s[16];
            tmem_ld16(tmem_s + lane_off + c0, s);
            const uint32_t vis = c0 < kc ? visible16(c0) : 0u;
#pragma unroll
            for (int j = 0; j < 16; ++j) s[j] = ((vis >> j) & 1u) ? fast_exp2(s[j] * p.scale_log2 - m_use) : 0.f;
#pragma unroll
            for (int gq = 0; gq < 2; ++gq) {
              uint32_t hi[4], lo[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int j = gq * 8 + 2 * e;
                l2[e & 1] += s[j] + s[j + 1];
                split2_pack(s[j], s[j + 1], hi[e], lo[e]);
              }
              const int c8 = ((c0 - rd * ROUND) >> 3) + gq;     // 8-key group within this round's 128 keys
              const int off = (c8 >> 3) * SUB + row * 128 + (((c8 & 7) ^ (row & 7)) << 4);
              *reinterpret_cast<uint4*>(As + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
              *reinterpret_cast<uint4*>(As + 2 * SUB + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
          }
          STACK_TRACE_POINT(7 + rd, cur_layer);
          if (rd == rounds - 1 && kc < kc_pad) {
            // value rows past the end of the cache meet p = 0, but 0 * garbage could still be NaN: clear them
            ok = wwait(&sc->bar_v, par);
            if (ok && eg == 0 && row < kc_pad - kc) {
#pragma unroll 1
              for (int sub = 0; sub < 2 * H2; ++sub)
#pragma unroll 1
                for (int i = 0; i < 8; ++i)
                  *reinterpret_cast<uint4*>(KVs + sub * KVSUB + (kc + row) * 128 + i * 16) = make_uint4(0, 0, 0, 0);
            }
          }
          if (ok) {
            fence_proxy_async_smem();
            mbar_arrive(&sc->bar_p[rd]);
          }
        }
        sc->red_sum[eg][row] = l2[0] + l2[1];
        STACK_TRACE_POINT(2, cur_layer);
        if (ok) ok = rounds == 2 ? wwait(&sc->bar_o[1], par2) : wwait(&sc->bar_o[0], par);
        STACK_TRACE_POINT(3, cur_layer);
        // Every thread holds 32 consecutive floats of its row per TMEM load and stores them straight to the partial
        // output: 128 contiguous bytes per thread, whole sectors.  (Staging the tile in shared memory so that a warp
        // writes whole rows cost two more barriers and a pass of index arithmetic, 3 us against 1.)
        if (ok) {                                               // warp-uniform: the TMEM load is a warp-wide instruction
          tc_fence_after();
          float4* dst = reinterpret_cast<float4*>(p.attO + out_row * DH);
#pragma unroll 1
          for (int c0 = eg * 32; c0 < DH; c0 += 64) {
            float o[32];
            tmem_ld32(tmem_o + lane_off + c0, o);
            if (row_valid) {
#pragma unroll
              for (int e = 0; e < 8; ++e) dst[(c0 >> 2) + e] = make_float4(o[4 * e], o[4 * e + 1], o[4 * e + 2], o[4 * e + 3]);
            }
          }
        }
        tc_fence_before();
        STACK_TRACE_POINT(9, cur_layer);
        worker_bar();                                           // both halves of every row's sum are in shared memory
        if (ok && row_valid && eg == 0) p.attML[out_row] = make_float2(m_row, sc->red_sum[0][row] + sc->red_sum[1][row]);
        STACK_TRACE_POINT(13, cur_layer);
        worker_bar();                                           // the staging area and red_* are free again
        if (wtid == 0) {
          __threadfence_block();
          *(volatile int*)&sc->units_done = au;                 // units this CTA has finished since the kernel began
        }
      }
    };

    // ---------------- merge of the key blocks, normalisation, hi / lo split for the O projection
    auto merge_step = [&]() {
      const size_t rows_alloc = (size_t)p.n_alloc * p.Hq;
      const int rows_total = p.n * p.Hq;
      const int n_splits = tab.splits;
      const size_t ao_plane = (size_t)p.n_alloc * p.q_dim;
      const int c = lane * 4;
#pragma unroll 1
      for (int r = cta * 8 + wwarp; r < rows_total; r += G * 8) {
        bf16* out = p.AO + (size_t)r * DH + c;
        const float2 none = make_float2(-INFINITY, 0.f);
        const float2 ml0 = lane < n_splits ? __ldcg(p.attML + (size_t)lane * rows_alloc + r) : none;
        const float2 ml1 = lane + 32 < n_splits ? __ldcg(p.attML + (size_t)(lane + 32) * rows_alloc + r) : none;
        constexpr int MB = 10;                        // partial outputs in flight per round trip to L2 (config 3 has 9 key blocks)
        float4 o[MB];
#pragma unroll
        for (int u = 0; u < MB; ++u)
          o[u] = (u < n_splits && c < DH) ? __ldcg(reinterpret_cast<const float4*>(p.attO + ((size_t)u * rows_alloc + r) * DH + c))
                                          : make_float4(0.f, 0.f, 0.f, 0.f);
        float mx = fmaxf(ml0.y > 0.f ? ml0.x : -INFINITY, ml1.y > 0.f ? ml1.x : -INFINITY);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
        const float w0 = ml0.y > 0.f ? exp2f(ml0.x - mx) : 0.f;
        const float w1 = ml1.y > 0.f ? exp2f(ml1.x - mx) : 0.f;
        float den = 0.f;                                 // terms added in block order: independent of timing
#pragma unroll 1
        for (int s = 0; s < n_splits; ++s) den += __shfl_sync(0xFFFFFFFFu, s < 32 ? ml0.y * w0 : ml1.y * w1, s & 31);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
        for (int s0 = 0; s0 < n_splits; s0 += MB) {
          if (s0 > 0) {
#pragma unroll
            for (int u = 0; u < MB; ++u) {
              const int s = s0 + u;
              o[u] = (s < n_splits && c < DH) ? __ldcg(reinterpret_cast<const float4*>(p.attO + ((size_t)s * rows_alloc + r) * DH + c))
                                              : make_float4(0.f, 0.f, 0.f, 0.f);
            }
          }
#pragma unroll
          for (int u = 0; u < MB; ++u) {
            const int s = s0 + u;
            float w = __shfl_sync(0xFFFFFFFFu, s < 32 ? w0 : w1, s & 31);
            if (s >= n_splits || !(w > 0.f)) {
              w = 0.f;
              o[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            acc.x += o[u].x * w; acc.y += o[u].y * w; acc.z += o[u].z * w; acc.w += o[u].w * w;
          }
        }
        if (c < DH) {
          const float rcp = 1.f / den;
          uint32_t ph[2], pl[2];
          split2_pack(acc.x * rcp, acc.y * rcp, ph[0], pl[0]);
          split2_pack(acc.z * rcp, acc.w * rcp, ph[1], pl[1]);
          *reinterpret_cast<uint2*>(out) = make_uint2(ph[0], ph[1]);
          *reinterpret_cast<uint2*>(out + ao_plane) = make_uint2(pl[0], pl[1]);
        }
      }
    };

    // ================= the sequence of steps
    const size_t stride_d = (size_t)p.n_alloc * p.d;
    const size_t stride_qkv = (size_t)p.n_alloc * p.qkv_dim;
#pragma unroll 1
    for (int sidx = 0; sidx < n_steps; ++sidx) {
      const int l = sidx / ST_PER_LAYER, st = sidx - l * ST_PER_LAYER;
      const bool head = l == p.n_layers;
      const int gk = gemm_kind_of(l, st, p.n_layers);
      cur_layer = l;
      int trace_kind = SPECASR_KIND_NORM;
      (void)trace_kind;
      STACK_TRACE_BEGIN();
      if (gk == ST_QKV || gk == ST_O || gk == ST_DOWN) {
        epi_partial(gemm_of(p, l, gk, cta, G), gk == ST_QKV ? stride_qkv : stride_d);
        trace_kind = gk == ST_QKV ? SPECASR_KIND_GEMM_QKV : gk == ST_O ? SPECASR_KIND_GEMM_O : SPECASR_KIND_GEMM_DOWN;
      } else if (gk == ST_GU || gk == -1) {
        wait_step(sidx - 1);                             // the row sums of squares of the norm before it
        STACK_TRACE_MARK();
        load_inv();
        epi_streamk(gemm_of(p, l, gk, cta, G), gk == ST_GU, p.epoch0 + 1 + l);
        trace_kind = gk == ST_GU ? SPECASR_KIND_GEMM_GU : SPECASR_KIND_GEMM_LM;
      } else if (st == ST_ATTN) {
        attention_step();
        worker_bar();
        if (wtid == 0) {
          __threadfence_block();
          *(volatile int*)&sc->attn_done = l + 1;
        }
        trace_kind = SPECASR_KIND_ATTN;
      } else {
        if (sidx > 0) wait_step(sidx - 1);               // every other step reads what the step before it wrote
        STACK_TRACE_MARK();
        if (st == ST_ROPE) {
          rope_step(l);
          trace_kind = SPECASR_KIND_ROPE;
        } else if (st == ST_MERGE) {
          merge_step();
          trace_kind = SPECASR_KIND_ATTN_MERGE;
        } else {                                         // a norm: attention, FFN or final
          const bool ffn = !head && st == ST_NORM2;
          norm_step(p.gains[head ? 2 * p.n_layers : 2 * l + (ffn ? 1 : 0)],
                    ffn ? p.splits_o : (sidx > 0 ? p.splits_down : 0), stride_d);
        }
      }
      arrive_step();
      STACK_TRACE_END(trace_kind, l);
    }
    (void)arrived;
  }

  tc_fence_before();
  __syncthreads();
  if (*abort) {
    // give copies still in flight time to land before the shared memory is handed back
#pragma unroll 1
    for (int i = 0; i < 64; ++i) __nanosleep(20000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

template <int DH>
cudaError_t launch_dh(const CUtensorMap& tmH, const CUtensorMap& tmAO, const CUtensorMap& tmA, const CUtensorMap& tmQ,
                      const SegTable& tab, const StackParams& p, int grid, size_t smem, cudaStream_t s) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(k_stack<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;           // all CTAs co-resident, or the launch fails
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_stack<DH>, tmH, tmAO, tmA, tmQ, tab, p);
}

}  // namespace

// Shapes the fused kernel covers: tensor-core attention (head_dim 64 / 128, pages of a multiple of 16 slots),
// up to 64 token rows (one activation box, both planes in one MMA), key-block count within one counter lane pair.
bool fused_stack_supported(const specasr_kv* wk, int n_total, bool att_tc, int splits) {
  const specasr_model* m = wk->m;
  if (m->cfg.gemm_path != 0 || !att_tc || !wk->attn_tc || m->w_maps_dev == nullptr) return false;
  if (n_total < 1 || n_total > 64) return false;
  if (splits > kMaxAttnSplits) return false;
  // every weight tile of a linear projection needs a CTA of its own
  const int groups_qkv = (m->qkv_dim + TM * TILE_M - 1) / (TM * TILE_M);
  const int groups_d = (m->cfg.d_model + TM * TILE_M - 1) / (TM * TILE_M);
  if (groups_qkv > m->n_sm || groups_d > m->n_sm) return false;
  return true;
}

size_t fused_stack_sync_bytes(const specasr_model* m) {
  return (((size_t)m->cfg.n_layers * ST_PER_LAYER + 2) * sizeof(int32_t) + 255) / 256 * 256;
}

bool launch_fused_stack(specasr_model* m, specasr_kv* wk, const SegTable& tab, int n_total, int n_max,
                        const int32_t* ctl_shared, bool want_head, float* out_logits, bool want_top2, cudaStream_t s) {
  const specasr_model_config& c = m->cfg;
  int n_pad = 16;
  while (n_pad < n_total) n_pad <<= 1;
  StackParams p;
  memset(&p, 0, sizeof(p));
  p.n_layers = c.n_layers; p.d = c.d_model; p.qkv_dim = m->qkv_dim; p.q_dim = m->q_dim;
  p.Hq = c.n_heads; p.Hkv = c.n_kv_heads; p.ffn = c.ffn; p.vocab = c.vocab; p.page_size = c.page_size;
  p.max_positions = c.max_positions;
  p.eps = c.rms_eps;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)c.head_dim);
  p.w_maps = m->w_maps_dev;
  p.gains = m->gains_dev;
  p.rope = m->rope_table;
  p.n = n_total; p.n_pad = n_pad; p.n_alloc = wk->n_alloc;
  p.stage_bytes = W_STAGE_BYTES + KSUB * n_pad * 2 * SUB_K * 2;
  const int epi_bytes = 2 * n_pad * 64 * 2;
  const int attn_bytes = 4 * SUB + 2 * (c.head_dim / 64) * KVSUB;
  int stages = (SMEM_LIMIT - (int)sizeof(StackCtl) - epi_bytes - 1024) / p.stage_bytes;
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  p.stages = stages;
  p.ring_bytes = stages * p.stage_bytes;
  if (p.ring_bytes < attn_bytes) p.ring_bytes = (attn_bytes + 1023) & ~1023;
  // k parts of the linear projections: tile groups * parts should just fill the SMs
  auto pick_splits = [&](int M, int K) {
    const int groups = (M + TM * TILE_M - 1) / (TM * TILE_M);
    const int KB = (K + KSUB * SUB_K - 1) / (KSUB * SUB_K);
    int sp = m->n_sm / groups;
    if (sp > kMaxSplitK) sp = kMaxSplitK;
    if (sp > KB) sp = KB;
    return sp < 1 ? 1 : sp;
  };
  p.splits_qkv = pick_splits(m->qkv_dim, c.d_model);
  p.splits_o = pick_splits(c.d_model, m->q_dim);
  p.splits_down = pick_splits(c.d_model, c.ffn);
  p.epoch0 = wk->gemm_epoch;
  wk->gemm_epoch += c.n_layers + 1;
  p.want_head = want_head ? 1 : 0;
  p.group = c.n_heads / c.n_kv_heads;
  p.nodes_per_tile = 128 / p.group;
  p.row_tiles = (n_max + p.nodes_per_tile - 1) / p.nodes_per_tile;
  p.attn_units = c.n_kv_heads * p.row_tiles * tab.count * tab.splits;
  p.ctl = const_cast<int32_t*>(ctl_shared);
  p.sync = wk->ws.sync;
  p.X = wk->ws.X; p.P = wk->ws.P; p.fixP = wk->ws.fixP; p.fixFlag = wk->ws.fixFlag;
  p.H = wk->ws.H; p.Q = wk->ws.Q; p.AO = wk->ws.AO; p.A = wk->ws.A;
  p.attO = wk->ws.attO; p.attML = wk->ws.attML; p.ssq = wk->ws.ssq; p.amax = wk->ws.amax;
  p.logits = out_logits;
  p.sec = want_top2 ? wk->ws.sec : nullptr;
  p.lse = want_top2 ? wk->ws.lse : nullptr;
  p.pos = wk->ws.pos; p.anc = wk->ws.anc;
#ifdef SPECASR_TRACE
  p.tr = wk->trace;
#endif
  const size_t smem = (size_t)p.ring_bytes + sizeof(StackCtl) + epi_bytes + 1024;
  int idx = 0;                                           // activation maps are indexed by log2(box rows / 16)
#pragma unroll 1
  for (int b = 16; b < n_pad; b <<= 1) ++idx;
  LaunchScope scope(wk, SPECASR_KIND_STACK, s);
  cudaError_t e = cudaMemsetAsync(wk->ws.sync, 0, fused_stack_sync_bytes(m), s);
  if (e == cudaSuccess) {
    if (c.head_dim == 64) e = launch_dh<64>(wk->tm_H[idx], wk->tm_AO[idx], wk->tm_A[idx], wk->tm_Q, tab, p, m->n_sm, smem, s);
    else e = launch_dh<128>(wk->tm_H[idx], wk->tm_AO[idx], wk->tm_A[idx], wk->tm_Q, tab, p, m->n_sm, smem, s);
  }
  if (e != cudaSuccess) {
    set_error("fused layer stack launch failed: %s", cudaGetErrorString(e));
    return false;
  }
  return true;
}
