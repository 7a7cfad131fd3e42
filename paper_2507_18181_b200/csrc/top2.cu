// specasr_top2_probs: the two most probable tokens of every row of a logits matrix and their softmax
// probabilities over the whole vocabulary -- the quantities the draft side of the method reads (Section IV-A:
// drafting stops where the normalised top-1 value falls below a threshold; Section IV-C: the second-ranked
// token at such a position seeds a side branch).  See include/specasr.h for the contract.
//
// One block per row.  Every thread scans a strided part of the row once, keeping its two largest packed
// (ordered logit, ~token id) keys and an online (max, sum of exp) pair; warps and then the block merge those.
#include "internal.h"
#include "device_utils.cuh"

namespace {

struct Top2 {
  unsigned long long a, b;     // a >= b, 0 = empty
};
__device__ __forceinline__ void top2_push(Top2& t, unsigned long long k) {
  if (k > t.a) {
    t.b = t.a;
    t.a = k;
  } else if (k > t.b) {
    t.b = k;
  }
}
__device__ __forceinline__ float key_value(unsigned long long k) {
  uint32_t u = (uint32_t)(k >> 32);
  u = (u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u;
  return __uint_as_float(u);
}
// (m, s) with s = sum of exp(x - m) over the elements seen so far; m = -inf and s = 0 when none
__device__ __forceinline__ void lse_merge(float& m, float& s, float m2, float s2) {
  const float mm = fmaxf(m, m2);
  if (mm == -INFINITY) return;
  s = s * expf(m - mm) + s2 * expf(m2 - mm);
  m = mm;
}

__global__ void __launch_bounds__(256) k_top2_probs(const float* __restrict__ logits, int vocab,
                                                    int32_t* __restrict__ out_ids, float* __restrict__ out_probs) {
  __shared__ Top2 s_top[8];
  __shared__ float s_m[8], s_s[8];
  grid_dep_launch();
  grid_dep_wait();
  const float* row = logits + (size_t)blockIdx.x * vocab;
  Top2 t{0ull, 0ull};
  float m = -INFINITY, s = 0.f;
  for (int v = threadIdx.x; v < vocab; v += 256) {
    const float x = row[v];
    top2_push(t, pack_max_key(x, (uint32_t)v));
    if (x > m) {
      s = s * expf(m - x) + 1.f;       // expf(-inf) = 0 covers the first element
      m = x;
    } else {
      s += expf(x - m);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long oa = __shfl_xor_sync(0xFFFFFFFFu, t.a, o), ob = __shfl_xor_sync(0xFFFFFFFFu, t.b, o);
    top2_push(t, oa);
    top2_push(t, ob);
    const float om = __shfl_xor_sync(0xFFFFFFFFu, m, o), os = __shfl_xor_sync(0xFFFFFFFFu, s, o);
    lse_merge(m, s, om, os);
  }
  const int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) {
    s_top[warp] = t;
    s_m[warp] = m;
    s_s[warp] = s;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) {
      top2_push(t, s_top[w].a);
      top2_push(t, s_top[w].b);
      lse_merge(m, s, s_m[w], s_s[w]);
    }
    if (t.b == 0ull) t.b = t.a;                    // a one-token vocabulary
    int32_t* ids = out_ids + (size_t)blockIdx.x * 2;
    float* pr = out_probs + (size_t)blockIdx.x * 2;
    ids[0] = (int32_t)(0xFFFFFFFFu - (uint32_t)(t.a & 0xFFFFFFFFull));
    ids[1] = (int32_t)(0xFFFFFFFFu - (uint32_t)(t.b & 0xFFFFFFFFull));
    pr[0] = expf(key_value(t.a) - m) / s;
    pr[1] = expf(key_value(t.b) - m) / s;
  }
}

}  // namespace

extern "C" specasr_status specasr_top2_probs(const float* logits, int32_t n_rows, int32_t vocab, int32_t* out_ids,
                                             float* out_probs, void* stream) {
  if (!logits || !out_ids || !out_probs) {
    set_error("specasr_top2_probs: null argument");
    return SPECASR_ERR_INVALID_ARG;
  }
  if (n_rows < 1 || vocab < 1) {
    set_error("specasr_top2_probs: n_rows = %d and vocab = %d must be positive", n_rows, vocab);
    return SPECASR_ERR_INVALID_ARG;
  }
  launch_pdl(k_top2_probs, dim3(n_rows), dim3(256), 0, (cudaStream_t)stream, logits, vocab, out_ids, out_probs);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    set_error("specasr_top2_probs: %s", cudaGetErrorString(e));
    return SPECASR_ERR_CUDA;
  }
  return SPECASR_OK;
}
