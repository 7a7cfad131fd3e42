// Tree-masked grouped-query attention over the paged KV cache, split over the KV axis.
//
// Node i sees every committed cache position [0, L) and those tree slots L + j for which j is i or an
// ancestor of i (bit j of the node's ancestor mask): this is the 2-D mask of a draft token tree.
// A CTA owns one KV head, a tile of 64 query rows (row = node * group + head-in-group, so the whole
// query group shares every K/V element that is staged) and one KV split; it stages K/V chunks of the
// split through shared memory with 16-byte loads, keeps an online softmax in base 2 and emits an
// unnormalised partial (max, sum, output) that k_attn_merge combines.
#include "internal.h"
#include "device_utils.cuh"

namespace {
constexpr int ROWS = 64;   // query rows per CTA
constexpr int KC = 32;     // keys per staged chunk

template <int DH>
__global__ void __launch_bounds__(256) k_tree_attention(const int32_t* __restrict__ ctl, const bf16* __restrict__ Q,
                                                        size_t q_plane_stride, const bf16* __restrict__ k_pool,
                                                        const bf16* __restrict__ v_pool,
                                                        const int32_t* __restrict__ page_table, int n_pages,
                                                        int page_size, int layer, int Hq, int Hkv, int n,
                                                        const unsigned long long* __restrict__ anc, int n_splits,
                                                        float scale_log2, float* __restrict__ attO,
                                                        float2* __restrict__ attML, size_t rows_alloc) {
  grid_dep_launch();
  grid_dep_wait();
  if (ctl[CTL_STATUS] != 0) return;
  extern __shared__ float smem[];
  float* Qs = smem;                         // [ROWS][DH + 1]
  float* Ks = Qs + ROWS * (DH + 1);         // [KC][DH + 1]
  float* Vs = Ks + KC * (DH + 1);           // [KC][DH]
  float* Ps = Vs + KC * DH;                 // [ROWS][KC + 1]

  const int tid = threadIdx.x;
  const int kvh = blockIdx.x;
  const int group = Hq / Hkv;
  const int rows_total = n * group;
  const int row0 = blockIdx.y * ROWS;
  const int split = blockIdx.z;
  const int L = ctl[CTL_LEN];
  const int Ltot = L + n;
  int chunk = (Ltot + n_splits - 1) / n_splits;
  chunk = (chunk + KC - 1) / KC * KC;
  const int k_begin = split * chunk;
  const int k_end = min(Ltot, k_begin + chunk);

  // stage the query tile (hi + lo -> fp32)
  constexpr int CH = DH / 8;
  for (int idx = tid; idx < ROWS * CH; idx += 256) {
    const int r = idx / CH, ch = idx % CH;
    const int rr = row0 + r;
    float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (rr < rows_total) {
      const int node = rr / group, qh = kvh * group + rr % group;
      const bf16* p = Q + ((size_t)node * Hq + qh) * DH + ch * 8;
      const uint4 h = *reinterpret_cast<const uint4*>(p);
      const uint4 l = *reinterpret_cast<const uint4*>(p + q_plane_stride);
      const uint32_t hw[4] = {h.x, h.y, h.z, h.w}, lw[4] = {l.x, l.y, l.z, l.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        v[2 * e] = bf16lo_to_f32(hw[e]) + bf16lo_to_f32(lw[e]);
        v[2 * e + 1] = bf16hi_to_f32(hw[e]) + bf16hi_to_f32(lw[e]);
      }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) Qs[r * (DH + 1) + ch * 8 + e] = v[e];
  }

  const int r = tid >> 2, kq = tid & 3;
  const int my_row = row0 + r;
  const int my_node = min(my_row, rows_total - 1) / group;
  unsigned long long my_anc[4];
#pragma unroll
  for (int w = 0; w < 4; ++w) my_anc[w] = anc[my_node * 4 + w];

  float m_run = -INFINITY, l_run = 0.f;
  float acc[DH / 4];
#pragma unroll
  for (int j = 0; j < DH / 4; ++j) acc[j] = 0.f;

  for (int c0 = k_begin; c0 < k_end; c0 += KC) {
    __syncthreads();   // previous chunk fully consumed (and Qs visible on the first pass)
    for (int idx = tid; idx < KC * CH; idx += 256) {
      const int kk = idx / CH, ch = idx % CH;
      const int kg = c0 + kk;
      float kv[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      float vv[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (kg < k_end) {
        const int page = page_table[kg / page_size];
        const size_t off = kv_plane_offset(layer, n_pages, Hkv, page_size, DH, page, kvh, 0) +
                           (size_t)(kg % page_size) * DH + ch * 8;
        const size_t plane = (size_t)page_size * DH;
        const uint4 kh = *reinterpret_cast<const uint4*>(k_pool + off);
        const uint4 kl = *reinterpret_cast<const uint4*>(k_pool + off + plane);
        const uint4 vh = *reinterpret_cast<const uint4*>(v_pool + off);
        const uint4 vl = *reinterpret_cast<const uint4*>(v_pool + off + plane);
        const uint32_t khw[4] = {kh.x, kh.y, kh.z, kh.w}, klw[4] = {kl.x, kl.y, kl.z, kl.w};
        const uint32_t vhw[4] = {vh.x, vh.y, vh.z, vh.w}, vlw[4] = {vl.x, vl.y, vl.z, vl.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          kv[2 * e] = bf16lo_to_f32(khw[e]) + bf16lo_to_f32(klw[e]);
          kv[2 * e + 1] = bf16hi_to_f32(khw[e]) + bf16hi_to_f32(klw[e]);
          vv[2 * e] = bf16lo_to_f32(vhw[e]) + bf16lo_to_f32(vlw[e]);
          vv[2 * e + 1] = bf16hi_to_f32(vhw[e]) + bf16hi_to_f32(vlw[e]);
        }
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        Ks[kk * (DH + 1) + ch * 8 + e] = kv[e];
        Vs[kk * DH + ch * 8 + e] = vv[e];
      }
    }
    __syncthreads();

    // scores of row r against keys kq, kq + 4, ...
    float s[KC / 4];
#pragma unroll
    for (int j = 0; j < KC / 4; ++j) s[j] = 0.f;
    for (int d = 0; d < DH; ++d) {
      const float qv = Qs[r * (DH + 1) + d];
#pragma unroll
      for (int j = 0; j < KC / 4; ++j) s[j] = fmaf(qv, Ks[(kq + 4 * j) * (DH + 1) + d], s[j]);
    }
    float cmax = -INFINITY;
#pragma unroll
    for (int j = 0; j < KC / 4; ++j) {
      const int kg = c0 + kq + 4 * j;
      bool vis = kg < L;
      if (!vis && kg < k_end) {
        const int t = kg - L;
        vis = (my_anc[t >> 6] >> (t & 63)) & 1ull;
      }
      s[j] = vis ? s[j] * scale_log2 : -INFINITY;
      cmax = fmaxf(cmax, s[j]);
    }
    cmax = fmaxf(cmax, __shfl_xor_sync(0xFFFFFFFFu, cmax, 1));
    cmax = fmaxf(cmax, __shfl_xor_sync(0xFFFFFFFFu, cmax, 2));
    const float m_new = fmaxf(m_run, cmax);
    float alpha = 1.f, psum = 0.f;
    if (m_new > -INFINITY) {
      alpha = exp2f(m_run - m_new);   // m_run = -inf gives 0
#pragma unroll
      for (int j = 0; j < KC / 4; ++j) {
        const float p = exp2f(s[j] - m_new);
        Ps[r * (KC + 1) + kq + 4 * j] = p;
        psum += p;
      }
    } else {
#pragma unroll
      for (int j = 0; j < KC / 4; ++j) Ps[r * (KC + 1) + kq + 4 * j] = 0.f;
    }
    psum += __shfl_xor_sync(0xFFFFFFFFu, psum, 1);
    psum += __shfl_xor_sync(0xFFFFFFFFu, psum, 2);
    l_run = l_run * alpha + psum;
    m_run = m_new;
    __syncwarp();   // the four threads of a row are in one warp; their P entries are now visible
#pragma unroll
    for (int j = 0; j < DH / 4; ++j) acc[j] *= alpha;
    for (int kk = 0; kk < KC; ++kk) {
      const float p = Ps[r * (KC + 1) + kk];
#pragma unroll
      for (int j = 0; j < DH / 4; ++j) acc[j] = fmaf(p, Vs[kk * DH + kq + 4 * j], acc[j]);
    }
  }

  if (my_row < rows_total) {
    const int qh = kvh * group + my_row % group;
    const size_t out_row = (size_t)split * rows_alloc + (size_t)my_node * Hq + qh;
#pragma unroll
    for (int j = 0; j < DH / 4; ++j) attO[out_row * DH + kq + 4 * j] = acc[j];
    if (kq == 0) attML[out_row] = make_float2(m_run, l_run);
  }
}

template <int DH>
void launch_dh(specasr_kv* kv, int layer, int n, int n_splits, cudaStream_t s) {
  const specasr_model* m = kv->m;
  const specasr_model_config& c = m->cfg;
  const int group = c.n_heads / c.n_kv_heads;
  const size_t smem = sizeof(float) * (ROWS * (DH + 1) + KC * (DH + 1) + KC * DH + ROWS * (KC + 1));
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(k_tree_attention<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    configured = true;
  }
  dim3 grid(c.n_kv_heads, (n * group + ROWS - 1) / ROWS, n_splits);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
  LaunchScope scope(kv, SPECASR_KIND_ATTN, s);
  launch_pdl(k_tree_attention<DH>, grid, dim3(256), smem, s, kv->ws.ctl, kv->ws.Q, (size_t)kv->n_alloc * m->q_dim, kv->k_pool,
                                               kv->v_pool, kv->page_table, kv->n_pages, c.page_size, layer,
                                               c.n_heads, c.n_kv_heads, n, kv->ws.anc, n_splits, scale_log2,
                                               kv->ws.attO, kv->ws.attML, (size_t)kv->n_alloc * c.n_heads);
}
}  // namespace

void launch_tree_attention(specasr_kv* kv, int layer, int n, int n_splits, cudaStream_t s) {
  switch (kv->m->cfg.head_dim) {
    case 32: launch_dh<32>(kv, layer, n, n_splits, s); break;
    case 64: launch_dh<64>(kv, layer, n, n_splits, s); break;
    default: launch_dh<128>(kv, layer, n, n_splits, s); break;
  }
}
