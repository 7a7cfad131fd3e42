// Small device helpers shared by the kernels.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

__device__ __forceinline__ float bf16lo_to_f32(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// x ~ hi + lo with hi = bf16(x), lo = bf16(x - hi): about 16 significant bits survive.
__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// 2^x by the special-function unit alone (relative error about 2^-22, denormal results flushed to zero).  exp2f()
// wraps the same instruction in range handling that the soft-max does not need (its arguments are <= 0 and a result
// below 2^-126 is as good as zero) and that made up a tenth of the attention step.
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Two values -> packed (hi0, hi1) and (lo0, lo1) words, element 0 in the low half; one packed
// conversion per plane.
__device__ __forceinline__ void split2_pack(float a, float b, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  const __nv_bfloat162 l = __floats2bfloat162_rn(a - bf16lo_to_f32(hi), b - bf16hi_to_f32(hi));
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// Sum over a 256-thread block; every thread receives the total.
__device__ __forceinline__ float block_sum_256(float v) {
  __shared__ float s_part[8];
  __shared__ float s_total;
  v = warp_sum(v);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x < 32) {
    float t = threadIdx.x < 8 ? s_part[threadIdx.x] : 0.f;
    t = warp_sum(t);
    if (threadIdx.x == 0) s_total = t;
  }
  __syncthreads();
  return s_total;
}

// Element offset of plane `plane` (0 = hi, 1 = lo) of (layer, physical page, kv head) in a KV pool
// laid out [n_layers][n_pages][n_kv_heads][2][page_size][head_dim].
__device__ __forceinline__ size_t kv_plane_offset(int layer, int n_pages, int Hkv, int page_size, int dh, int page,
                                                  int kvh, int plane) {
  return ((((size_t)layer * n_pages + page) * Hkv + kvh) * 2 + plane) * (size_t)page_size * dh;
}

// Weight matrices [M, K] are stored tile-packed: 128-row x 64-column tiles, each 16 KB contiguous (row-major inside),
// ordered [row tile][column tile]; K is padded to a multiple of 128 columns and M to a multiple of 128 rows with
// zeros.  A pipeline stage of the projections (128 rows x 128 columns) is then one contiguous 32 KB run in HBM.
__host__ __device__ __forceinline__ int packed_col_tiles(int K) { return 2 * ((K + 127) / 128); }
__host__ __device__ __forceinline__ size_t packed_weight_offset(int m, int k, int K) {
  return ((((size_t)(m >> 7) * packed_col_tiles(K) + (k >> 6)) * 128 + (m & 127)) << 6) + (k & 63);
}

// Order-preserving map of a float to an unsigned key, packed with the complement of an index so that
// a plain unsigned max picks the largest value and, among equals, the lowest index.
__device__ __forceinline__ unsigned long long pack_max_key(float v, uint32_t idx) {
  uint32_t u = __float_as_uint(v);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - idx);
}

// One trace record per thread block (see TraceBuf): construct at kernel entry, mark() after the wait for the
// previous kernel, the destructor stamps the end.  Only the library variant built with -DSPECASR_TRACE carries
// it (through the SPECASR_TRACE_* macros): even switched off, the extra parameter and live value changed the
// register allocation of several kernels and cost the step about 2 %.
#ifdef SPECASR_TRACE
struct TraceScope {
  unsigned long long* e;
  __device__ __forceinline__ static unsigned long long now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
  }
  __device__ __forceinline__ TraceScope(const TraceBuf& tr, int kind) : e(nullptr) {
    if (tr.buf != nullptr && threadIdx.x == 0 && threadIdx.y == 0 && threadIdx.z == 0) {
      const unsigned long long slot = atomicAdd(tr.buf, 1ull);
      if (slot < tr.cap) {
        e = tr.buf + 2 + slot * 4;
        e[0] = (unsigned long long)kind;
        e[1] = now();
        e[2] = 0;
        e[3] = 0;
      }
    }
  }
  __device__ __forceinline__ void mark() {
    if (e) e[3] = now();
  }
  __device__ __forceinline__ ~TraceScope() {
    if (e) e[2] = now();
  }
};
#endif

// Programmatic dependent launch (see launch_pdl): wait for the previous kernel of the stream, and let
// the next one begin its prologue.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Rows of the fused QKV weight are stored in rotary-paired order within each head: row 32 g + j holds
// feature 16 g + j and row 32 g + 16 + j its rotation partner dh/2 further on (0 <= j < 16).
__device__ __forceinline__ int qkv_row_of_feature(int e, int dh) {
  const int half = dh >> 1;
  const int k = e % half;
  return ((k >> 4) << 5) | ((e / half) << 4) | (k & 15);
}
