// Weight-streaming projections on the 5th-generation tensor cores (sm_100a).
//
//   D[m][t] = sum_k W[m][k] * (hi[t][k] + lo[t][k])        W: [M, K] bf16, activations: two bf16 planes
//
// The weight matrix is the MMA "A" operand (128 rows per tile), the tree tokens are the MMA "N"
// dimension, so a 64-node tree costs one 128 x 64 fp32 accumulator per tile and every weight byte is
// read from HBM exactly once.  Both operands are K-major and arrive by TMA into 128-byte-swizzled
// shared-memory tiles.  The hi and lo activation planes sit back to back in shared memory and form ONE
// MMA of N = 2 x tokens (the weight tile, the large operand, is fetched once for both); the epilogue
// adds the two halves of the accumulator.
// A pipeline stage holds one k-block of `tm` adjacent weight tiles and the matching activation block,
// so with tm = 2 the activation bytes (which every CTA re-reads from L2) are half the weight bytes.
// From 128 tokens on the two planes are "folded": one MMA per plane (N = tokens of the box), both accumulating
// into the same TMEM columns, so a tile costs n instead of 2 n columns and two accumulator sets of 256 tokens
// fit the 512 columns.
//
// Scheduling.  The kernel is persistent, at most one CTA per SM, over (tile group, k-block) units.
//  - Linear outputs (QKV, O, down): the k-blocks of every tile group are cut into `splits` equal
//    parts, one CTA each; a CTA writes its fp32 partial sums to plane `split` and the consumer kernel
//    adds the planes in a fixed order.
//  - Non-linear epilogues (gate/up with SiLU * up, LM head with arg-max): the units of the whole
//    matrix are cut into equal contiguous ranges, one per CTA, so every SM streams the same number of
//    weight bytes whatever the tile count.  A tile group whose k-blocks fall into two ranges is summed
//    in a fixed order: the CTA holding its later k-blocks (which it processes first) parks its partial
//    sums in a workspace slot and publishes a flag; the CTA holding k-block 0 (which it processes
//    last) adds them in CTA order and runs the epilogue.  All CTAs are co-resident and every flag wait
//    is bounded.
//
// Roles: warp 0 issues TMA, one thread of warp 1 issues tcgen05.mma, warps 2..9 drain TMEM
// (tcgen05.ld; warps w and w + 4 share a lane quadrant and take alternate 16-token blocks) into the epilogue; two TMEM accumulator sets let the epilogue of one tile group overlap
// the main loop of the next.
//
// Programmatic dependent launch: the weight tiles of the first pipeline stages are requested before
// the kernel waits for its predecessor in the stream, since weights never change; only activation
// loads and global writes come after that wait.
//
// Every mbarrier or flag wait is bounded by wall-clock time; on expiry the CTA records
// SPECASR_ERR_TIMEOUT in the status word, lets copies in flight land, frees its TMEM and returns.
#include "internal.h"
#include "device_utils.cuh"
#include "sm100_ptx.cuh"

using namespace sm100;

namespace {

constexpr int TILE_M = 128;
constexpr int SUB_K = 64;             // bf16 elements = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int W_SUB_BYTES = TILE_M * SUB_K * 2;
constexpr int MAX_STAGES = 6;
constexpr int SMEM_LIMIT = 227 * 1024;  // dynamic shared memory one CTA may ask for

struct alignas(16) SharedCtl {
  unsigned long long full[MAX_STAGES];
  unsigned long long empty[MAX_STAGES];
  unsigned long long acc_full[2];
  unsigned long long acc_empty[2];
  unsigned long long key[SPECASR_MAX_NODES];
  uint32_t tmem_base;
  int abort;
};

struct TcParams {
  int M, K, n, n_pad, n_alloc, box_rows, stages, ksub, tm, n_buf, tmem_cols, KB, tiles, groups, splits, epoch;
  int kt64;                 // 64-column tiles per row tile of the packed weight matrix
  int fold;                 // launch the FOLD instantiation: hi and lo products share the TMEM columns
  int32_t* ctl;
  float* fixP;              // [grid][tm][n_pad][128] parked partial sums (hi + lo halves added) of split tile groups
  int32_t* fixFlag;         // [grid] launch number of the partial sums each CTA parked last
  float* P;                 // EPI_PARTIAL: [splits][n_alloc][M]
  bf16* A;                  // EPI_SWIGLU: [2][n_alloc][M/2]
  unsigned long long* amax; // EPI_ARGMAX: [tiles][n_alloc]
  float* logits;            // EPI_ARGMAX: optional [n][M]
#ifdef SPECASR_TRACE
  TraceBuf tr;
  int kind;                 // SPECASR_KIND_* of this launch
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
constexpr int EPI_THREADS = 256;      // warps 2..9
__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

template <int EPI, bool FOLD>
__global__ void __launch_bounds__(64 + EPI_THREADS, 1) k_proj(const __grid_constant__ CUtensorMap tmW,
                                                 const __grid_constant__ CUtensorMap tmAct, TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  SPECASR_TRACE_SCOPE(p.tr, p.kind);
  uint8_t* tiles = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int w_bytes = p.tm * p.ksub * W_SUB_BYTES;
  const int act_sub = p.n_pad * 2 * SUB_K * 2;         // both planes of one 64-wide k sub-block
  const int stage_bytes = w_bytes + p.ksub * act_sub;
  SharedCtl* sc = (SharedCtl*)(tiles + (size_t)p.stages * stage_bytes);
  bf16* epi_stage = (bf16*)(sc + 1);                    // EPI_SWIGLU: [2 planes][<= 64 tokens][64] output tile

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = gridDim.x, cta = blockIdx.x;
  const int KB = p.KB;
  const long long U = (long long)p.groups * KB;
  long long u0, u1;
  if (EPI == EPI_PARTIAL) {           // one tile group, one part of its k-blocks
    const int group = cta / p.splits, split = cta % p.splits;
    u0 = (long long)group * KB + (long long)split * KB / p.splits;
    u1 = (long long)group * KB + (long long)(split + 1) * KB / p.splits;
  } else {                            // equal contiguous ranges of the whole unit list
    u0 = cta * U / G;
    u1 = (cta + 1) * U / G;
  }
  const int n_blocks = p.n_pad / p.box_rows;
  const int tile_cols = FOLD ? p.n_pad : 2 * p.n_pad;   // TMEM columns of one tile: hi | lo halves unless folded
  const int acc_cols = p.tm * tile_cols;                // one accumulator set

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&sc->full[s], 1);
      mbar_init(&sc->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sc->acc_full[b], 1);
      mbar_init(&sc->acc_empty[b], EPI_THREADS);
    }
    sc->abort = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmW);
    tma_prefetch_desc(&tmAct);
  }
  if (warp == 1) tmem_alloc(&sc->tmem_base, (uint32_t)p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_launch_dependents();
  const uint32_t tmem_base = sc->tmem_base;
  volatile int* abort = &sc->abort;
  int32_t* status = p.ctl + CTL_STATUS;

  if (warp == 0 && lane == 0) {
    // ---------------- TMA producer
    const int total = (int)(u1 - u0);
    auto load_w = [&](int i) {
      const long long u = u0 + i;
      const int group = (int)(u / KB), kb = (int)(u % KB), s = i % p.stages;
      uint8_t* st = tiles + (size_t)s * stage_bytes;
      for (int t = 0; t < p.tm; ++t)       // rows past M are the zero padding of the packed matrix
        for (int q = 0; q < p.ksub; ++q)
          tma_load_2d(st + (t * p.ksub + q) * W_SUB_BYTES, &tmW, 0,
                      ((group * p.tm + t) * p.kt64 + kb * p.ksub + q) * TILE_M, &sc->full[s]);   // tile-packed weights
    };
    auto load_act = [&](int i) {
      const int kb = (int)((u0 + i) % KB), s = i % p.stages;
      uint8_t* st = tiles + (size_t)s * stage_bytes + w_bytes;
      for (int q = 0; q < p.ksub; ++q)
        for (int jb = 0; jb < n_blocks; ++jb)
          tma_load_3d(st + q * act_sub + (size_t)jb * p.box_rows * 2 * SUB_K * 2, &tmAct, (kb * p.ksub + q) * SUB_K,
                      jb * p.box_rows, 0, &sc->full[s]);
    };
    // weights never change: request the first stages before waiting for the previous kernel
    const int pre = total < p.stages ? total : p.stages;
    for (int i = 0; i < pre; ++i) {
      mbar_expect_tx(&sc->full[i], (uint32_t)stage_bytes);
      load_w(i);
    }
    pdl_wait();
    SPECASR_TRACE_MARK();
    if (*(volatile int32_t*)status != 0) {
      if (pre > 0) *abort = 1;       // weight tiles are in flight: hold the shared memory until they land
    } else {
      for (int i = 0; i < pre; ++i) load_act(i);
      for (int i = pre; i < total; ++i) {
        const int s = i % p.stages;
        const uint32_t ph = (uint32_t)(i / p.stages) & 1u;
        if (!mbar_wait(&sc->empty[s], ph ^ 1u, abort, status)) break;
        mbar_expect_tx(&sc->full[s], (uint32_t)stage_bytes);
        load_w(i);
        load_act(i);
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer
    pdl_wait();
    if (*(volatile int32_t*)status == 0) {
      // both planes of a token block in one MMA of N = 2 * box rows, or (folded) one MMA per plane into the same columns
      const uint32_t idesc = make_idesc_bf16(FOLD ? p.box_rows : 2 * p.box_rows);
      int i = 0, seg = 0;
      bool ok = true;
      for (long long u = u0; u < u1 && ok; ++seg) {
        const int kb0 = (int)(u % KB);
        const int kb1 = (int)((u1 - u) < (long long)(KB - kb0) ? kb0 + (u1 - u) : KB);
        const int b = seg % p.n_buf;
        if (!mbar_wait(&sc->acc_empty[b], (uint32_t)((seg / p.n_buf) & 1) ^ 1u, abort, status)) break;
        tc_fence_after();
        const uint32_t d_base = tmem_base + (uint32_t)(b * acc_cols);
        for (int kb = kb0; kb < kb1; ++kb, ++i) {
          const int s = i % p.stages;
          const uint32_t ph = (uint32_t)(i / p.stages) & 1u;
          if (!mbar_wait(&sc->full[s], ph, abort, status)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t w_addr = smem_u32(tiles + (size_t)s * stage_bytes);
          const uint32_t act_addr = w_addr + w_bytes;
          for (int t = 0; t < p.tm; ++t) {
            for (int q = 0; q < p.ksub; ++q) {
              const uint32_t a_lo = smem_desc_lo(w_addr + (t * p.ksub + q) * W_SUB_BYTES);
              for (int jb = 0; jb < n_blocks; ++jb) {
                const uint32_t b_addr = act_addr + q * act_sub + (uint32_t)(jb * 2 * p.box_rows * SUB_K * 2);
                const uint32_t d_addr = d_base + (uint32_t)(t * tile_cols + jb * (FOLD ? 1 : 2) * p.box_rows);
                const uint32_t b_lo = smem_desc_lo(b_addr);
                const uint32_t lo_lo = smem_desc_lo(b_addr + (uint32_t)(p.box_rows * SUB_K * 2));   // lo rows follow the hi rows
#pragma unroll
                for (int k = 0; k < SUB_K / UMMA_K; ++k) {
                  const uint32_t acc = k > 0 ? 1u : ((kb > kb0 || q > 0) ? 1u : 0u);
                  umma_bf16_lo(d_addr, a_lo + ((k * UMMA_K * 2) >> 4), b_lo + ((k * UMMA_K * 2) >> 4), idesc, acc);
                  if (FOLD) umma_bf16_lo(d_addr, a_lo + ((k * UMMA_K * 2) >> 4), lo_lo + ((k * UMMA_K * 2) >> 4), idesc, 1u);
                }
              }
            }
          }
          umma_commit(&sc->empty[s]);   // arrives once these MMAs have read the stage
        }
        if (ok) umma_commit(&sc->acc_full[b]);
        u += kb1 - kb0;
      }
    }
  } else if (warp >= 2) {
    // ---------------- epilogue: TMEM lane = output row of the tile
    pdl_wait();
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int etid = threadIdx.x - 64;
    const int c_first = ((warp - 2) >> 2) * 16;          // this warp's first 16-token block; the stride is 32
    bool ok = *(volatile int32_t*)status == 0;
    int seg = 0;
    // value of token block [c0, c0 + 16) of tile t2: hi half + lo half of the accumulator
    auto load16 = [&](uint32_t lane_addr, int t2, int c0, float* v) {
      if (FOLD) {
        tmem_ld16(lane_addr + (uint32_t)(t2 * p.n_pad + c0), v);
        return;
      }
      const uint32_t col = (uint32_t)(t2 * 2 * p.n_pad + (c0 / p.box_rows) * 2 * p.box_rows + c0 % p.box_rows);
      float lo[16];
      tmem_ld16x2(lane_addr + col, lane_addr + col + (uint32_t)p.box_rows, v, lo);
#pragma unroll
      for (int j = 0; j < 16; ++j) v[j] += lo[j];
    };
    for (long long u = u0; u < u1; ++seg) {
      const int group = (int)(u / KB);
      const int kb0 = (int)(u % KB);
      const int kb1 = (int)((u1 - u) < (long long)(KB - kb0) ? kb0 + (u1 - u) : KB);
      u += kb1 - kb0;
      const int b = seg % p.n_buf;
      // A CTA that holds the first k-blocks of a split tile group adds the partial sums parked by the CTAs
      // that hold the rest.  Those were parked early in their run, so their flags are polled and the first
      // tile's parked sums are requested here, while this segment's MMAs are still running.
      int last = cta;
      if (EPI != EPI_PARTIAL && kb0 == 0 && kb1 != KB)
        while (last + 1 < G && (last + 1) * U / G < (long long)(group + 1) * KB) ++last;
      const bool quick = p.n_pad <= 64;          // at most two 16-token blocks per warp and tile: keep them in registers
      float pk0[16], pk1[16];
      auto load_parked = [&](int t2, int c0, float* f) {
#pragma unroll
        for (int j = 0; j < 16; ++j) f[j] = 0.f;
        if (c0 < p.n_pad)
          for (int cc = cta + 1; cc <= last; ++cc) {
            const float* src = p.fixP + ((size_t)(cc * p.tm + t2) * p.n_pad + c0) * TILE_M + row;
#pragma unroll
            for (int j = 0; j < 16; ++j) f[j] += __ldcg(src + j * TILE_M);
          }
      };
      if (last > cta) {
        if (ok && threadIdx.x == 64) {
          const unsigned long long t0 = global_ns();
          for (int cc = cta + 1; cc <= last && !*abort; ++cc) {
            while (ld_acquire(p.fixFlag + cc) != p.epoch) {
              if (*abort) break;
              if (global_ns() - t0 > WAIT_LIMIT_NS) {
                *abort = 1;
                atomicExch(status, (int32_t)SPECASR_ERR_TIMEOUT);
                break;
              }
              __nanosleep(64);
            }
          }
        }
        epi_bar();
        if (*abort) ok = false;
        if (ok && quick) {
          load_parked(0, c_first, pk0);
          load_parked(0, c_first + 32, pk1);
        }
      }
      if (ok) ok = mbar_wait_relaxed(&sc->acc_full[b], (uint32_t)((seg / p.n_buf) & 1), abort, status);
      tc_fence_after();
      const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(b * acc_cols);

      if (EPI == EPI_PARTIAL) {
        if (ok) {
          float* out = p.P + (size_t)(cta % p.splits) * p.n_alloc * p.M;
          for (int t2 = 0; t2 < p.tm; ++t2) {
            const int m = (group * p.tm + t2) * TILE_M + row;
            for (int c0 = c_first; c0 < p.n_pad; c0 += 32) {
              float v[16];
              load16(lane_addr, t2, c0, v);
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (c0 + j < p.n && m < p.M) out[(size_t)(c0 + j) * p.M + m] = v[j];
            }
          }
          tc_fence_before();
          mbar_arrive(&sc->acc_empty[b]);
        }
        continue;
      }

      if (kb0 != 0) {
        // later k-blocks of a tile group whose first k-blocks belong to an earlier CTA: park the partial sums
        float* dst = p.fixP + (size_t)cta * p.tm * p.n_pad * TILE_M;
        if (ok) {
          for (int t2 = 0; t2 < p.tm; ++t2)
            for (int c0 = c_first; c0 < p.n_pad; c0 += 32) {
              float v[16];
              load16(lane_addr, t2, c0, v);
#pragma unroll
              for (int j = 0; j < 16; ++j) dst[(size_t)(t2 * p.n_pad + c0 + j) * TILE_M + row] = v[j];
            }
          tc_fence_before();
          mbar_arrive(&sc->acc_empty[b]);
          __threadfence();
        }
        epi_bar();
        if (ok && threadIdx.x == 64) st_release(p.fixFlag + cta, p.epoch);
        continue;
      }

      // first k-blocks of the tile group (or all of them): run the epilogue on the complete sums
      for (int t2 = 0; t2 < p.tm; ++t2) {
        const int tile = group * p.tm + t2;
        if (tile >= p.tiles) break;
        const int m = tile * TILE_M + row;
        const bool row_ok = m < p.M;
        if (EPI == EPI_ARGMAX) {
          for (int t = etid; t < SPECASR_MAX_NODES; t += EPI_THREADS) sc->key[t] = 0ull;
          epi_bar();
        }
        // the SwiGLU output of 128 tokens or more is staged in shared memory 64 tokens at a time
        constexpr bool CHUNKED = FOLD && EPI == EPI_SWIGLU;      // folded launches have at least 128 tokens
        const int tok_chunk = CHUNKED ? 64 : p.n_pad;
        for (int tc0 = 0; tc0 < (CHUNKED ? p.n_pad : 1); tc0 += tok_chunk) {
          if (ok) {
            // parked sums of this tile (requested a tile ahead); the next tile's are requested now
            float cur0[16], cur1[16];
            if (last > cta && quick) {
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                cur0[j] = pk0[j];
                cur1[j] = pk1[j];
              }
              if (t2 + 1 < p.tm) {
                load_parked(t2 + 1, c_first, pk0);
                load_parked(t2 + 1, c_first + 32, pk1);
              }
            }
            for (int c0 = tc0 + c_first; c0 < tc0 + tok_chunk; c0 += 32) {
              float v[16];
              load16(lane_addr, t2, c0, v);
              if (last > cta) {
                if (quick) {
                  const bool first = c0 == c_first;
#pragma unroll
                  for (int j = 0; j < 16; ++j) v[j] += first ? cur0[j] : cur1[j];
                } else {
                  float f[16];
                  load_parked(t2, c0, f);
#pragma unroll
                  for (int j = 0; j < 16; ++j) v[j] += f[j];
                }
              }
              if (EPI == EPI_SWIGLU) {
                // rows 2f / 2f + 1 of the tile are gate / up of feature f: the even lane keeps the hi plane of
                // the product, the odd lane the lo plane, staged in shared memory for 16-byte global stores
                float a[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  const float other = __shfl_xor_sync(0xFFFFFFFFu, v[j], 1);
                  const float g = (lane & 1) ? other : v[j];
                  const float up = (lane & 1) ? v[j] : other;
                  a[j] = __fdividef(g, 1.f + __expf(-g)) * up;
                }
                bf16* st = epi_stage + (size_t)(lane & 1) * tok_chunk * 64 + (size_t)(c0 - tc0) * 64 + (row >> 1);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  bf16 hi, lo;
                  split_bf16(a[j], hi, lo);
                  st[j * 64] = (lane & 1) ? lo : hi;
                }
              } else if (EPI == EPI_ARGMAX) {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  const int t = c0 + j;
                  if (p.logits && t < p.n && row_ok) p.logits[(size_t)t * p.M + m] = v[j];
                  // warp arg-max: largest ordered key, then the lowest row among its holders
                  uint32_t key = __float_as_uint(v[j]);
                  key = (key & 0x80000000u) ? ~key : (key | 0x80000000u);
                  if (!row_ok) key = 0u;
                  const uint32_t best = __reduce_max_sync(0xFFFFFFFFu, key);
                  const uint32_t who = __reduce_min_sync(0xFFFFFFFFu, key == best ? (uint32_t)m : 0xFFFFFFFFu);
                  if (lane == 0 && t < p.n && best != 0u)
                    atomicMax(&sc->key[t], ((unsigned long long)best << 32) | (unsigned long long)(0xFFFFFFFFu - who));
                }
              }
            }
          }
          if (EPI == EPI_SWIGLU) {
            epi_bar();
            if (ok) {
              const int F = p.M >> 1;
              const int f0 = tile * 64;
              int nt = p.n - tc0;                             // tokens of this chunk that exist
              nt = nt < 0 ? 0 : (nt > tok_chunk ? tok_chunk : nt);
              const int chunks = 2 * nt * 8;                  // 16-byte pieces of the [2][nt][64] tile
              for (int idx = etid; idx < chunks; idx += EPI_THREADS) {
                const int plane = idx / (nt * 8), rem = idx % (nt * 8);
                const int t = rem >> 3, ch = rem & 7;
                if (f0 + ch * 8 < F)
                  *reinterpret_cast<uint4*>(p.A + (size_t)plane * p.n_alloc * F + (size_t)(tc0 + t) * F + f0 + ch * 8) =
                      *reinterpret_cast<const uint4*>(epi_stage + (size_t)plane * tok_chunk * 64 + t * 64 + ch * 8);
              }
            }
            epi_bar();
          }
        }
        if (EPI == EPI_ARGMAX) {
          epi_bar();
          if (ok)
            for (int t = etid; t < p.n; t += EPI_THREADS) p.amax[(size_t)tile * p.n_alloc + t] = sc->key[t];
        }
      }
      if (ok) {
        tc_fence_before();
        mbar_arrive(&sc->acc_empty[b]);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort) {
    // give copies still in flight time to land before the shared memory is handed back
    for (int i = 0; i < 64; ++i) __nanosleep(20000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}



int pick_box_rows(int n_pad) {
  int b = 128;      // one MMA spans both planes of a box: N = 2 * box rows <= 256
  while (b > 16 && (n_pad % b) != 0) b >>= 1;
  return b;
}

template <int EPI, bool FOLD>
void launch_epi(const CUtensorMap& tmW, const CUtensorMap& tmAct, const TcParams& p, int grid, size_t smem,
                cudaStream_t s) {
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(k_proj<EPI, FOLD>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT);
    configured = true;
  }
  launch_pdl(k_proj<EPI, FOLD>, dim3(grid), dim3(64 + EPI_THREADS), smem, s, tmW, tmAct, p);
}

}  // namespace

bool make_tensor_map_2d(CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer, uint32_t box_inner,
                        uint32_t box_outer) {
  EncodeTiledFn enc = get_encode();
  if (!enc) {
    set_error("cuTensorMapEncodeTiled is not available from this driver");
    return false;
  }
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {inner * 2};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_error("cuTensorMapEncodeTiled failed with code %d (inner %llu, outer %llu)", (int)r,
              (unsigned long long)inner, (unsigned long long)outer);
    return false;
  }
  return true;
}

bool make_tensor_map_nd(CUtensorMap* out, const void* base, int rank, const uint64_t* dims, const uint64_t* strides,
                        const uint32_t* box) {
  EncodeTiledFn enc = get_encode();
  if (!enc) {
    set_error("cuTensorMapEncodeTiled is not available from this driver");
    return false;
  }
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], es[5];
  for (int i = 0; i < rank; ++i) {
    d[i] = dims[i];
    b[i] = box[i];
    es[i] = 1;
    if (i + 1 < rank) st[i] = strides[i];
  }
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_error("cuTensorMapEncodeTiled (rank %d) failed with code %d", rank, (int)r);
    return false;
  }
  return true;
}

// Activation planes [2][n_alloc][K]: box = (64 columns, box_rows rows, both planes).
bool make_act_map(CUtensorMap* out, const void* base, uint64_t K, uint64_t n_alloc, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) {
    set_error("cuTensorMapEncodeTiled is not available from this driver");
    return false;
  }
  cuuint64_t dims[3] = {K, n_alloc, 2};
  cuuint64_t strides[2] = {K * 2, n_alloc * K * 2};
  cuuint32_t box[3] = {64, box_rows, 2};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_error("cuTensorMapEncodeTiled (activations) failed with code %d", (int)r);
    return false;
  }
  return true;
}

int gemm_tc_tiles(int M) { return (M + TILE_M - 1) / TILE_M; }

// Tile groups per stage and k sub-blocks per stage for trees padded to n_pad nodes.
static void tc_shape(int n_pad, int* tm, int* ksub) {
  // One weight tile per stage: with 64 tokens a stage is 64 KB and three stages fit, which measured faster
  // than two stages of a tile pair (tm = 2, activation block shared by both tiles) although the pair halves
  // the activation traffic; the kernel keeps tm as a parameter.
  // From 128 tokens on the hi / lo products are folded into one accumulator, which keeps two accumulator sets
  // within the 512 TMEM columns up to 256 tokens (the epilogue of one tile overlaps the next tile's main loop).
  // A tile pair per stage (tm = 2) was measured there as well: it halves the activation bytes per weight byte
  // but leaves only two 96 KB stages at 256 tokens, and the step is bound by the latency of a stage, not by
  // bandwidth (256 tokens, gate/up: 175 us with pairs, 144 us without).
  *tm = 1;
  *ksub = n_pad <= 64 ? 2 : 1;                    // two 16 KB tiles of the packed matrix per stage: 32 KB contiguous
}

// Number of k parts of the linear projections: tile groups * parts should just fill the SMs.
int gemm_tc_pick_splits(const specasr_model* m, int M, int K, int n_pad) {
  int tm, ksub;
  tc_shape(n_pad, &tm, &ksub);
  const int groups = (gemm_tc_tiles(M) + tm - 1) / tm;
  const int KB = (K + ksub * SUB_K - 1) / (ksub * SUB_K);
  int s = m->n_sm / groups;
  if (s > kMaxSplitK) s = kMaxSplitK;
  if (s > KB) s = KB;
  if (s < 1) s = 1;
  return s;
}

// Bytes of the parked-partial workspace for trees of up to n_alloc nodes.
size_t gemm_tc_fixup_bytes(const specasr_model* m, int n_alloc) {
  return (size_t)m->n_sm * 2 * n_alloc * TILE_M * sizeof(float);
}

void launch_gemm_tc(specasr_kv* kv, const GemmArgs& a, int kind, cudaStream_t s) {
  const specasr_model* m = kv->m;
  TcParams p;
  memset(&p, 0, sizeof(p));
  p.M = a.M; p.K = a.K; p.n = a.n; p.n_pad = a.n_pad; p.n_alloc = a.n_alloc;
  p.box_rows = pick_box_rows(a.n_pad);
  tc_shape(a.n_pad, &p.tm, &p.ksub);
  const int stage_bytes = p.ksub * (p.tm * W_SUB_BYTES + a.n_pad * 2 * SUB_K * 2);
  p.fold = a.n_pad >= 128 ? 1 : 0;
  const int epi_bytes = a.epilogue == EPI_SWIGLU ? 2 * (a.n_pad < 64 ? a.n_pad : 64) * 64 * 2 : 0;   // staged output tile
  int stages = (SMEM_LIMIT - (int)sizeof(SharedCtl) - epi_bytes - 1024) / stage_bytes;
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  p.stages = stages;
  const int acc_cols = p.tm * (p.fold ? 1 : 2) * a.n_pad;
  p.n_buf = 2 * acc_cols <= 512 ? 2 : 1;
  int cols = 32;
  while (cols < p.n_buf * acc_cols) cols <<= 1;
  p.tmem_cols = cols;
  p.KB = (a.K + p.ksub * SUB_K - 1) / (p.ksub * SUB_K);
  p.kt64 = packed_col_tiles(a.K);
  p.tiles = gemm_tc_tiles(a.M);
  p.groups = (p.tiles + p.tm - 1) / p.tm;
  p.splits = a.epilogue == EPI_PARTIAL ? a.splits : 0;
  p.epoch = ++kv->gemm_epoch;
  p.ctl = const_cast<int32_t*>(a.ctl);
  p.fixP = kv->ws.fixP;
  p.fixFlag = kv->ws.fixFlag;
  p.P = a.P; p.A = a.A; p.amax = a.amax; p.logits = a.logits;
#ifdef SPECASR_TRACE
  p.tr = kv->trace;
  p.kind = kind;
#endif
  const long long units = (long long)p.groups * p.KB;
  const int grid = a.epilogue == EPI_PARTIAL ? p.groups * p.splits : (int)(units < m->n_sm ? units : m->n_sm);
  const size_t smem = (size_t)stages * stage_bytes + sizeof(SharedCtl) + epi_bytes + 1024;
  int idx = 0;      // a.tmAct is an array of maps indexed by log2(box_rows / 16)
  for (int b = 16; b < p.box_rows; b <<= 1) ++idx;
  const CUtensorMap& act = a.tmAct[idx];
  LaunchScope scope(kv, kind, s);
  if (p.fold) {
    switch (a.epilogue) {
      case EPI_PARTIAL: launch_epi<EPI_PARTIAL, true>(*a.tmW, act, p, grid, smem, s); break;
      case EPI_SWIGLU: launch_epi<EPI_SWIGLU, true>(*a.tmW, act, p, grid, smem, s); break;
      default: launch_epi<EPI_ARGMAX, true>(*a.tmW, act, p, grid, smem, s); break;
    }
  } else {
    switch (a.epilogue) {
      case EPI_PARTIAL: launch_epi<EPI_PARTIAL, false>(*a.tmW, act, p, grid, smem, s); break;
      case EPI_SWIGLU: launch_epi<EPI_SWIGLU, false>(*a.tmW, act, p, grid, smem, s); break;
      default: launch_epi<EPI_ARGMAX, false>(*a.tmW, act, p, grid, smem, s); break;
    }
  }
}
