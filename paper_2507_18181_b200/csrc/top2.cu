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

// The same two tokens and probabilities from what the vocabulary projection's epilogue left per 128-row tile
// (best and second-best packed key, max and sum of exp): one block per node, threads stride over the tiles.
__global__ void __launch_bounds__(256) k_top2_from_tiles(const __grid_constant__ SegTable tab,
                                                         const int32_t* __restrict__ ctl_shared,
                                                         const unsigned long long* __restrict__ first,
                                                         const unsigned long long* __restrict__ second,
                                                         const float2* __restrict__ lse, int n_tiles, int n_alloc,
                                                         int32_t* __restrict__ out_ids, float* __restrict__ out_probs) {
  __shared__ Top2 s_top[8];
  __shared__ float s_m[8], s_s[8];
  grid_dep_launch();
  grid_dep_wait();
  const int node = blockIdx.x;
  int b = 0;
  while (b + 1 < tab.count && node >= tab.seg[b].row0 + tab.seg[b].n) ++b;
  int32_t* ids = out_ids + (size_t)node * 2;
  float* pr = out_probs + (size_t)node * 2;
  if (tab.seg[b].ctl[CTL_STATUS] != 0 || (ctl_shared && ctl_shared[CTL_STATUS] != 0)) {
    if (threadIdx.x == 0) {
      ids[0] = ids[1] = -1;
      pr[0] = pr[1] = 0.f;
    }
    return;
  }
  Top2 t{0ull, 0ull};
  float m = -INFINITY, s = 0.f;
  for (int tile = threadIdx.x; tile < n_tiles; tile += 256) {
    top2_push(t, __ldcg(first + (size_t)tile * n_alloc + node));
    top2_push(t, __ldcg(second + (size_t)tile * n_alloc + node));
    const float2 ms = __ldcg(lse + (size_t)tile * n_alloc + node);
    lse_merge(m, s, ms.x, ms.y);
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
    ids[0] = (int32_t)(0xFFFFFFFFu - (uint32_t)(t.a & 0xFFFFFFFFull));
    ids[1] = (int32_t)(0xFFFFFFFFu - (uint32_t)(t.b & 0xFFFFFFFFull));
    pr[0] = expf(key_value(t.a) - m) / s;
    pr[1] = expf(key_value(t.b) - m) / s;
  }
}

}  // namespace

void launch_top2_from_tiles(specasr_kv* wk, const SegTable& t, const int32_t* ctl_shared, int n_total, int n_tiles,
                            int32_t* out_ids, float* out_probs, cudaStream_t s) {
  LaunchScope scope(wk, SPECASR_KIND_ACCEPT, s);
  launch_pdl(k_top2_from_tiles, dim3(n_total), dim3(256), 0, s, t, ctl_shared, wk->ws.amax, wk->ws.sec, wk->ws.lse, n_tiles,
             wk->n_alloc, out_ids, out_probs);
}

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
