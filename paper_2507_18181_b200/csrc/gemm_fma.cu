// Plain FMA projections: out[t][m] = sum_k W[m][k] * (hi[t][k] + lo[t][k]), fp32 accumulation.
// This path exists to cross-check the tensor-core projections on a GPU (same operands, same
// epilogues, different engine); the product path does not dispatch to it.
#include "internal.h"
#include "device_utils.cuh"

namespace {
constexpr int BM = 64, BN = 64, BK = 16;

template <int EPI>
__global__ void __launch_bounds__(256) k_gemm_fma(GemmArgs a) {
  grid_dep_launch();
  grid_dep_wait();
  if (a.ctl[CTL_STATUS] != 0) return;
  __shared__ float Ws[BK][BM + 4];
  __shared__ float As[BK][BN + 4];
  __shared__ unsigned long long s_key[BN];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.x * BM, t0 = blockIdx.y * BN;
  const bf16* act_hi = a.act;
  const bf16* act_lo = a.act + (size_t)a.n_alloc * a.K;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  if (EPI == EPI_ARGMAX && tid < BN) s_key[tid] = 0ull;

  const int lr = tid >> 2, lk = (tid & 3) * 4;
  for (int k0 = 0; k0 < a.K; k0 += BK) {
    float w[4] = {0.f, 0.f, 0.f, 0.f}, x[4] = {0.f, 0.f, 0.f, 0.f};
    if (m0 + lr < a.M && k0 + lk < a.K) {
      const uint2 v = *reinterpret_cast<const uint2*>(a.W + packed_weight_offset(m0 + lr, k0 + lk, a.K));
      w[0] = bf16lo_to_f32(v.x); w[1] = bf16hi_to_f32(v.x);
      w[2] = bf16lo_to_f32(v.y); w[3] = bf16hi_to_f32(v.y);
    }
    if (t0 + lr < a.n && k0 + lk < a.K) {
      const size_t off = (size_t)(t0 + lr) * a.K + k0 + lk;
      const uint2 h = *reinterpret_cast<const uint2*>(act_hi + off);
      const uint2 l = *reinterpret_cast<const uint2*>(act_lo + off);
      x[0] = bf16lo_to_f32(h.x) + bf16lo_to_f32(l.x); x[1] = bf16hi_to_f32(h.x) + bf16hi_to_f32(l.x);
      x[2] = bf16lo_to_f32(h.y) + bf16lo_to_f32(l.y); x[3] = bf16hi_to_f32(h.y) + bf16hi_to_f32(l.y);
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      Ws[lk + j][lr] = w[j];
      As[lk + j][lr] = x[j];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 wv = *reinterpret_cast<const float4*>(&Ws[kk][ty * 4]);
      const float4 xv = *reinterpret_cast<const float4*>(&As[kk][tx * 4]);
      const float wr[4] = {wv.x, wv.y, wv.z, wv.w};
      const float xr[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(wr[i], xr[j], acc[i][j]);
    }
  }

  const int m = m0 + ty * 4;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int t = t0 + tx * 4 + j;
    if (EPI == EPI_PARTIAL) {
      if (t < a.n)
        for (int i = 0; i < 4; ++i)
          if (m + i < a.M) a.P[(size_t)t * a.M + m + i] = acc[i][j];
    } else if (EPI == EPI_SWIGLU) {
      if (t < a.n) {
        const int F = a.M / 2;
        for (int i = 0; i < 4; i += 2) {
          if (m + i + 1 < a.M) {
            const float g = acc[i][j], u = acc[i + 1][j];
            const float v = g / (1.f + expf(-g)) * u;
            bf16 hi, lo;
            split_bf16(v, hi, lo);
            const size_t o = (size_t)t * F + (m + i) / 2;
            a.A[o] = hi;
            a.A[(size_t)a.n_alloc * F + o] = lo;
          }
        }
      }
    } else {
      if (t < a.n) {
        unsigned long long best = 0ull;
        for (int i = 0; i < 4; ++i) {
          if (m + i < a.M) {
            if (a.logits) a.logits[(size_t)t * a.M + m + i] = acc[i][j];
            const unsigned long long key = pack_max_key(acc[i][j], (uint32_t)(m + i));
            best = key > best ? key : best;
          }
        }
        atomicMax(&s_key[tx * 4 + j], best);
      }
    }
  }
  if (EPI == EPI_ARGMAX) {
    __syncthreads();
    if (tid < BN && t0 + tid < a.n) a.amax[(size_t)blockIdx.x * a.n_alloc + t0 + tid] = s_key[tid];
  }
}
}  // namespace

int gemm_fma_tiles(int M) { return (M + BM - 1) / BM; }

void launch_gemm_fma(specasr_kv* kv, const GemmArgs& a, int kind, cudaStream_t s) {
  LaunchScope scope(kv, kind, s);
  dim3 grid((a.M + BM - 1) / BM, (a.n + BN - 1) / BN);
  if (a.epilogue == EPI_PARTIAL) launch_pdl(k_gemm_fma<EPI_PARTIAL>, grid, dim3(256), 0, s, a);
  else if (a.epilogue == EPI_SWIGLU) launch_pdl(k_gemm_fma<EPI_SWIGLU>, grid, dim3(256), 0, s, a);
  else launch_pdl(k_gemm_fma<EPI_ARGMAX>, grid, dim3(256), 0, s, a);
}
