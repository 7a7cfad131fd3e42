// Weight-streaming projections on the 5th-generation tensor cores (sm_100a).
//
//   D[m][t] = sum_k W[m][k] * (hi[t][k] + lo[t][k])        W: [M, K] bf16, activations: two bf16 planes
//
// The weight matrix is the MMA "A" operand (M = 128 rows per CTA tile), the tree tokens are the MMA
// "N" dimension, so a 64-node tree costs one 128 x 64 accumulator per tile and every weight byte is
// read from HBM exactly once.  Both operands are K-major and arrive by TMA into 128-byte-swizzled
// shared-memory tiles; the hi and lo activation planes are two MMAs into the same TMEM accumulator.
// One warp issues TMA, one thread issues tcgen05.mma, four warps drain TMEM (tcgen05.ld) into the
// fused epilogue.  Grid = (M tiles, K splits): split-K planes are summed by the consumer kernel in a
// fixed order, which keeps the result deterministic.
//
// Every mbarrier wait is bounded by wall-clock time; on expiry the CTA records SPECASR_ERR_TIMEOUT in
// the status word, lets copies in flight land, frees its TMEM and returns.
#include "internal.h"
#include "device_utils.cuh"
#include "sm100_ptx.cuh"

#include <stdio.h>

using namespace sm100;

namespace {

constexpr int TILE_M = 128;
constexpr int TILE_K = 64;            // bf16 elements = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int W_TILE_BYTES = TILE_M * TILE_K * 2;
constexpr int MAX_STAGES = 8;
constexpr int SMEM_BUDGET = 200 * 1024;

struct SharedCtl {
  unsigned long long full[MAX_STAGES];
  unsigned long long empty[MAX_STAGES];
  unsigned long long accum;
  unsigned long long key[SPECASR_MAX_NODES];
  uint32_t tmem_base;
  int abort;
};

struct TcParams {
  int M, K, n, n_pad, n_alloc, box_rows, stages, tmem_cols, splits;
  float* P;
  bf16* A;
  unsigned long long* amax;
  float* logits;
  int32_t* ctl;
};

template <int EPI>
__global__ void __launch_bounds__(192, 1) k_gemm_tc(const __grid_constant__ CUtensorMap tmW,
                                                    const __grid_constant__ CUtensorMap tmAct, TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  if (p.ctl[CTL_STATUS] != 0) return;
  uint8_t* tiles = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int act_bytes = p.n_pad * 2 * TILE_K * 2;     // both planes
  const int stage_bytes = W_TILE_BYTES + act_bytes;
  SharedCtl* sc = (SharedCtl*)(tiles + (size_t)p.stages * stage_bytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, split = blockIdx.y;
  const int KB = (p.K + TILE_K - 1) / TILE_K;
  const int kb0 = (int)(((long long)split * KB) / p.splits);
  const int kb1 = (int)(((long long)(split + 1) * KB) / p.splits);
  const int n_blocks = p.n_pad / p.box_rows;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&sc->full[s], 1);
      mbar_init(&sc->empty[s], 1);
    }
    mbar_init(&sc->accum, 1);
    sc->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (EPI == EPI_ARGMAX)
    for (int t = threadIdx.x; t < SPECASR_MAX_NODES; t += blockDim.x) sc->key[t] = 0ull;
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sc->tmem_base)),
                 "r"((uint32_t)p.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = sc->tmem_base;
  volatile int* abort = &sc->abort;
  int32_t* status = p.ctl + CTL_STATUS;

  if (warp == 0 && lane == 0) {
    // ---------------- TMA producer
    int it = 0;
    for (int kb = kb0; kb < kb1; ++kb, ++it) {
      const int s = it % p.stages;
      const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
      if (!mbar_wait(&sc->empty[s], ph ^ 1u, abort, status)) break;
      uint8_t* st = tiles + (size_t)s * stage_bytes;
      mbar_expect_tx(&sc->full[s], (uint32_t)stage_bytes);
      tma_load_2d(st, &tmW, kb * TILE_K, tile * TILE_M, &sc->full[s]);
      for (int jb = 0; jb < n_blocks; ++jb)
        tma_load_3d(st + W_TILE_BYTES + (size_t)jb * p.box_rows * 2 * TILE_K * 2, &tmAct, kb * TILE_K,
                    jb * p.box_rows, 0, &sc->full[s]);
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer
    const uint32_t idesc = make_idesc_bf16(p.box_rows);
    int it = 0;
    bool ok = true;
    for (int kb = kb0; kb < kb1; ++kb, ++it) {
      const int s = it % p.stages;
      const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
      if (!mbar_wait(&sc->full[s], ph, abort, status)) {
        ok = false;
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t w_addr = smem_u32(tiles + (size_t)s * stage_bytes);
      const uint32_t act_addr = w_addr + W_TILE_BYTES;
      for (int jb = 0; jb < n_blocks; ++jb) {
        for (int plane = 0; plane < 2; ++plane) {
          const uint32_t b_addr = act_addr + (uint32_t)((jb * 2 + plane) * p.box_rows * TILE_K * 2);
#pragma unroll
          for (int k = 0; k < TILE_K / UMMA_K; ++k) {
            const uint64_t ad = make_smem_desc(w_addr + k * UMMA_K * 2);
            const uint64_t bd = make_smem_desc(b_addr + k * UMMA_K * 2);
            const uint32_t acc = (kb > kb0 || plane > 0 || k > 0) ? 1u : 0u;
            umma_bf16(tmem_base + (uint32_t)(jb * p.box_rows), ad, bd, idesc, acc);
          }
        }
      }
      umma_commit(&sc->empty[s]);   // arrives once these MMAs have read the stage
    }
    if (ok) umma_commit(&sc->accum);
  } else if (warp >= 2) {
    // ---------------- epilogue: TMEM lane = output row of the tile
    const int quad = warp & 3;
    const int m = tile * TILE_M + quad * 32 + lane;
    const bool row_ok = m < p.M;
    if (mbar_wait(&sc->accum, 0u, abort, status)) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
      for (int c0 = 0; c0 < p.n_pad; c0 += 16) {
        float v[16];
        tmem_ld16(lane_addr + (uint32_t)c0, v);
        if (EPI == EPI_PARTIAL) {
          float* out = p.P + (size_t)split * p.n_alloc * p.M;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int t = c0 + j;
            if (t < p.n && row_ok) out[(size_t)t * p.M + m] = v[j];
          }
        } else if (EPI == EPI_SWIGLU) {
          const int F = p.M >> 1;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int t = c0 + j;
            const float other = __shfl_xor_sync(0xFFFFFFFFu, v[j], 1);
            const float g = (lane & 1) ? other : v[j];
            const float u = (lane & 1) ? v[j] : other;
            const float a = g / (1.f + expf(-g)) * u;
            bf16 hi, lo;
            split_bf16(a, hi, lo);
            if (t < p.n && row_ok) {
              const size_t o = (size_t)t * F + (m >> 1);
              if (lane & 1) p.A[(size_t)p.n_alloc * F + o] = lo;
              else p.A[o] = hi;
            }
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int t = c0 + j;
            if (p.logits && t < p.n && row_ok) p.logits[(size_t)t * p.M + m] = v[j];
            unsigned long long key = row_ok ? pack_max_key(v[j], (uint32_t)m) : 0ull;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, key, o);
              key = other > key ? other : key;
            }
            if (lane == 0 && t < p.n) atomicMax(&sc->key[t], key);
          }
        }
      }
      if (EPI == EPI_ARGMAX) {
        asm volatile("bar.sync 1, 128;" ::: "memory");
        for (int t = threadIdx.x - 64; t < p.n; t += 128) p.amax[(size_t)tile * p.n_alloc + t] = sc->key[t];
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (*abort) {
    // give copies still in flight time to land before the shared memory is handed back
    for (int i = 0; i < 64; ++i) __nanosleep(20000);
    __syncthreads();
  }
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols)
                 : "memory");
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
  int b = 256;
  while (b > 16 && (n_pad % b) != 0) b >>= 1;
  return b;
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

int gemm_tc_pick_splits(const specasr_model* m, int M, int K) {
  const int tiles = gemm_tc_tiles(M);
  const int KB = (K + TILE_K - 1) / TILE_K;
  int s = m->n_sm / tiles;
  if (s > kMaxSplitK) s = kMaxSplitK;
  if (s > KB) s = KB;
  if (s < 1) s = 1;
  return s;
}

void launch_gemm_tc(specasr_kv* kv, const GemmArgs& a, int kind, cudaStream_t s) {
  TcParams p;
  p.M = a.M; p.K = a.K; p.n = a.n; p.n_pad = a.n_pad; p.n_alloc = a.n_alloc;
  p.box_rows = pick_box_rows(a.n_pad);
  const int stage_bytes = W_TILE_BYTES + a.n_pad * 2 * TILE_K * 2;
  int stages = (SMEM_BUDGET - (int)sizeof(SharedCtl) - 1024) / stage_bytes;
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  p.stages = stages;
  int cols = 32;
  while (cols < a.n_pad) cols <<= 1;
  p.tmem_cols = cols;
  p.splits = a.epilogue == EPI_PARTIAL ? a.splits : 1;
  p.P = a.P; p.A = a.A; p.amax = a.amax; p.logits = a.logits;
  p.ctl = const_cast<int32_t*>(a.ctl);
  const size_t smem = (size_t)stages * stage_bytes + sizeof(SharedCtl) + 1024;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(k_gemm_tc<EPI_PARTIAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET);
    cudaFuncSetAttribute(k_gemm_tc<EPI_SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET);
    cudaFuncSetAttribute(k_gemm_tc<EPI_ARGMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET);
    configured = true;
  }
  const CUtensorMap* act = &a.tmAct[0];
  // a.tmAct points at an array of maps indexed by log2(box_rows / 16)
  int idx = 0;
  for (int b = 16; b < p.box_rows; b <<= 1) ++idx;
  act = &a.tmAct[idx];
  dim3 grid(gemm_tc_tiles(a.M), p.splits);
  LaunchScope scope(kv, kind, s);
  if (a.epilogue == EPI_PARTIAL) k_gemm_tc<EPI_PARTIAL><<<grid, 192, smem, s>>>(*a.tmW, *act, p);
  else if (a.epilogue == EPI_SWIGLU) k_gemm_tc<EPI_SWIGLU><<<grid, 192, smem, s>>>(*a.tmW, *act, p);
  else k_gemm_tc<EPI_ARGMAX><<<grid, 192, smem, s>>>(*a.tmW, *act, p);
}
