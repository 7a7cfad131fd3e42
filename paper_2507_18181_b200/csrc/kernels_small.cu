// Integer and element-wise kernels of the verification step: tree preparation, embedding gather,
// RMSNorm with operand split, rotary embedding + KV append, attention merge, accept, commit.
#include <cooperative_groups.h>

#include "internal.h"
#include "device_utils.cuh"

// ------------------------------------------------------------------------------------------------
// Tree preparation: validates the parent array, derives depth, position and the ancestor-or-self
// bitmask of every node (the rows of the 2-D tree attention mask), and sets the status word that
// every later kernel of the call checks.
// One block per utterance of the call; tokens / parent / depth / pos / anc are indexed by workspace row.
__global__ void k_tree_prep(const __grid_constant__ SegTable tab, const int32_t* __restrict__ tokens,
                            const int32_t* __restrict__ parent, int vocab, int32_t* __restrict__ depth,
                            int32_t* __restrict__ pos, unsigned long long* __restrict__ anc SPECASR_TRACE_PARAM) {
  __shared__ int s_bad;
  __shared__ int s_parent[SPECASR_MAX_NODES];     // the ancestor walk would otherwise be a chain of global loads
  SPECASR_TRACE_SCOPE(tr, SPECASR_KIND_PREP);
  const int i = threadIdx.x;
  const SegDev& sg = tab.seg[blockIdx.x];
  int32_t* ctl = sg.ctl;
  const int n = sg.n, capacity = sg.capacity;
  if (tokens) tokens += sg.row0;
  parent += sg.row0;
  depth += sg.row0;
  pos += sg.row0;
  anc += (size_t)sg.row0 * 4;
  grid_dep_launch();
  grid_dep_wait();
  SPECASR_TRACE_MARK();
  if (i == 0) s_bad = 0;
  __syncthreads();
  const int L = ctl[CTL_LEN];
  if (i < n) {
    const int p = parent[i];
    s_parent[i] = p;
    const int t = tokens ? tokens[i] : 0;
    const bool bad = (i == 0 ? p != -1 : (p < 0 || p >= i)) || t < 0 || t >= vocab;
    if (bad) atomicOr(&s_bad, 1);
  }
  if (i == 0 && (L < 0 || L + n > capacity)) atomicOr(&s_bad, 2);
  __syncthreads();
  if (s_bad) {
    if (i == 0) ctl[CTL_STATUS] = (s_bad & 1) ? SPECASR_ERR_INVALID_TREE : SPECASR_ERR_KV_CAPACITY;
    return;
  }
  if (i < n) {
    unsigned long long m[4] = {0ull, 0ull, 0ull, 0ull};
    int d = 0;
    int j = i;
    // parent[j] < j was checked above, so the walk ends after at most i + 1 steps
    while (j >= 0 && d <= n) {
      m[j >> 6] |= 1ull << (j & 63);
      j = s_parent[j];
      ++d;
    }
    depth[i] = d - 1;
    pos[i] = L + d - 1;
#pragma unroll
    for (int w = 0; w < 4; ++w) anc[i * 4 + w] = m[w];
  }
  if (i == 0) {
    ctl[CTL_STATUS] = SPECASR_OK;
    ctl[CTL_N] = n;
  }
}

// Context fill: a chunk of n consecutive positions is a chain, i.e. plain causal attention.
// Only the first chunk of a context-fill call starts from a clean status: a chunk that was refused (capacity, a
// token id outside the vocabulary) keeps every later chunk of the same call from running on top of the gap.
__global__ void k_chain_prep(int32_t* __restrict__ ctl, int n, int capacity, int first, int32_t* __restrict__ depth,
                             int32_t* __restrict__ pos, unsigned long long* __restrict__ anc) {
  const int i = threadIdx.x;
  grid_dep_launch();
  grid_dep_wait();
  if (!first && ctl[CTL_STATUS] != 0) return;
  const int L = ctl[CTL_LEN];
  if (L < 0 || L + n > capacity) {
    if (i == 0) ctl[CTL_STATUS] = SPECASR_ERR_KV_CAPACITY;
    return;
  }
  if (i < n) {
    depth[i] = i;
    pos[i] = L + i;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const int lo = w * 64;
      unsigned long long m = 0ull;
      if (i >= lo + 63) m = ~0ull;
      else if (i >= lo) m = (2ull << (i - lo)) - 1ull;
      anc[i * 4 + w] = m;
    }
  }
  if (i == 0) {
    ctl[CTL_STATUS] = SPECASR_OK;
    ctl[CTL_N] = n;
  }
}

void launch_tree_prep(specasr_kv* wk, const SegTable& t, const int32_t* tokens, const int32_t* parent, cudaStream_t s) {
  LaunchScope scope(wk, SPECASR_KIND_PREP, s);
  launch_pdl(k_tree_prep, dim3(t.count), dim3(256), 0, s, t, tokens, parent, wk->m->cfg.vocab, wk->ws.depth,
             wk->ws.pos, wk->ws.anc SPECASR_TRACE_ARG(wk));
}

void launch_chain_prep(specasr_kv* kv, int n, bool first, cudaStream_t s) {
  const specasr_model* m = kv->m;
  int cap = kv->max_pages * m->cfg.page_size;
  if (m->cfg.max_positions < cap) cap = m->cfg.max_positions;
  LaunchScope scope(kv, SPECASR_KIND_PREP, s);
  launch_pdl(k_chain_prep, dim3(1), dim3(256), 0, s, kv->ws.ctl, n, cap, first ? 1 : 0, kv->ws.depth, kv->ws.pos, kv->ws.anc);
}

// ------------------------------------------------------------------------------------------------
// Layer-0 inputs: embedding rows (bf16 -> fp32 residual stream), or caller-provided vectors.
// The utterance that owns workspace row `row` (segments are laid out back to back in table order).
__device__ __forceinline__ int segment_of_row(const SegTable& tab, int row) {
  int b = 0;
  while (b + 1 < tab.count && row >= tab.seg[b].row0 + tab.seg[b].n) ++b;
  return b;
}

// A token id outside [0, vocab) is never turned into an address: the row is skipped and the utterance's status
// word is set, which turns the rest of the call into no-ops (tree verification has checked the ids before; a
// context fill has not).
__global__ void k_embed_tokens(const __grid_constant__ SegTable tab, const int32_t* __restrict__ tokens,
                               const bf16* __restrict__ E, int d, int vocab, float* __restrict__ X SPECASR_TRACE_PARAM) {
  grid_dep_launch();
  SPECASR_TRACE_SCOPE(tr, SPECASR_KIND_PREP);
  grid_dep_wait();
  SPECASR_TRACE_MARK();
  const int i = blockIdx.x;
  int32_t* ctl = tab.seg[segment_of_row(tab, i)].ctl;
  if (ctl[CTL_STATUS] != 0) return;
  const int tok = tokens[i];
  if (tok < 0 || tok >= vocab) {
    if (threadIdx.x == 0) ctl[CTL_STATUS] = SPECASR_ERR_INVALID_TREE;
    return;
  }
  const bf16* row = E + (size_t)tok * d;
  float* x = X + (size_t)i * d;
  for (int k = threadIdx.x * 8; k < d; k += blockDim.x * 8) {
    const uint4 v = *reinterpret_cast<const uint4*>(row + k);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float4 a, b;
    a.x = bf16lo_to_f32(w[0]); a.y = bf16hi_to_f32(w[0]);
    a.z = bf16lo_to_f32(w[1]); a.w = bf16hi_to_f32(w[1]);
    b.x = bf16lo_to_f32(w[2]); b.y = bf16hi_to_f32(w[2]);
    b.z = bf16lo_to_f32(w[3]); b.w = bf16hi_to_f32(w[3]);
    *reinterpret_cast<float4*>(x + k) = a;
    *reinterpret_cast<float4*>(x + k + 4) = b;
  }
}

__global__ void k_copy_embeds(const int32_t* __restrict__ ctl, const float* __restrict__ src, int d,
                              float* __restrict__ X) {
  grid_dep_launch();
  grid_dep_wait();
  if (ctl[CTL_STATUS] != 0) return;
  const int i = blockIdx.x;
  for (int k = threadIdx.x * 4; k < d; k += blockDim.x * 4)
    *reinterpret_cast<float4*>(X + (size_t)i * d + k) = *reinterpret_cast<const float4*>(src + (size_t)i * d + k);
}

void launch_embed_tokens(specasr_kv* wk, const SegTable& t, int n_total, const int32_t* tokens, cudaStream_t s) {
  LaunchScope scope(wk, SPECASR_KIND_PREP, s);
  launch_pdl(k_embed_tokens, dim3(n_total), dim3(128), 0, s, t, tokens, wk->m->embed, wk->m->cfg.d_model,
             wk->m->cfg.vocab, wk->ws.X SPECASR_TRACE_ARG(wk));
}

void launch_copy_embeds(specasr_kv* kv, const float* embeds, int n, cudaStream_t s) {
  LaunchScope scope(kv, SPECASR_KIND_PREP, s);
  launch_pdl(k_copy_embeds, dim3(n), dim3(128), 0, s, kv->ws.ctl, embeds, kv->m->cfg.d_model, kv->ws.X);
}

// ------------------------------------------------------------------------------------------------
// RMSNorm with the residual update folded in: x <- x + sum of the previous projection's partial planes
// (fixed order, hence deterministic), h = x * rsqrt(mean(x^2) + eps) * g, emitted as two bf16 planes
// hi = bf16(h), lo = bf16(h - hi) so that the tensor-core projections see ~16 significant bits of every
// activation.  Rows n..n_pad-1 of both planes are zeroed.
// A cluster of four CTAs owns a row, one quarter each, so that the few megabytes of partial planes are
// pulled through 4 x n SMs at once and every thread has all its loads (x and up to 12 planes) in flight
// together: an in-order core would otherwise pay one L2 round trip per plane.  The four partial sums of
// squares meet through distributed shared memory (each CTA writes its own into all four) and are added in rank
// order.  (Two CTAs per row, i.e. at most
// one block per SM at 64 rows, measured the same.)
constexpr int kNormCluster = 4;

template <int ITER>
__global__ void __launch_bounds__(256) k_rmsnorm_split(const int32_t* __restrict__ ctl, float* __restrict__ X,
                                                       const float* __restrict__ P, int n_partials,
                                                       size_t partial_stride, const float* __restrict__ gain,
                                                       int d, int d_part, float eps, int n, size_t plane_stride,
                                                       bf16* __restrict__ H SPECASR_TRACE_PARAM) {
  namespace cg = cooperative_groups;
  __shared__ float s_ss[kNormCluster];
  grid_dep_launch();
  SPECASR_TRACE_SCOPE(tr, SPECASR_KIND_NORM);
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int row = blockIdx.x / kNormCluster;
  const int tid = threadIdx.x;
  const int k_end = min(d, (rank + 1) * d_part);
  int kk[ITER];
  float4 g[ITER];
#pragma unroll
  for (int it = 0; it < ITER; ++it) {        // gains never change: fetch them before waiting
    kk[it] = rank * d_part + (it * 256 + tid) * 4;
    g[it] = kk[it] < k_end ? *reinterpret_cast<const float4*>(gain + kk[it]) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  grid_dep_wait();
  SPECASR_TRACE_MARK();
  const int status = row < n ? 0 : ctl[CTL_STATUS];   // rows that exist read it behind their data loads (below)
  if (status != 0) return;                   // same for the whole cluster
  bf16* hi = H + (size_t)row * d;
  bf16* lo = hi + plane_stride;
  if (row >= n) {                            // same for the whole cluster
#pragma unroll
    for (int it = 0; it < ITER; ++it)
      if (kk[it] < k_end) {
        *reinterpret_cast<uint2*>(hi + kk[it]) = make_uint2(0, 0);
        *reinterpret_cast<uint2*>(lo + kk[it]) = make_uint2(0, 0);
      }
    return;
  }
  float* x = X + (size_t)row * d;
  float4 v[ITER];
#pragma unroll
  for (int it = 0; it < ITER; ++it)
    v[it] = kk[it] < k_end ? *reinterpret_cast<const float4*>(x + kk[it]) : make_float4(0.f, 0.f, 0.f, 0.f);
  const int late_status = ctl[CTL_STATUS];   // requested behind the row's data instead of in front of it
  constexpr int BATCH = ITER == 1 ? kMaxSplitK : (ITER == 2 ? 6 : 3);
  for (int s0 = 0; s0 < n_partials; s0 += BATCH) {
    float4 q[BATCH][ITER];
#pragma unroll
    for (int u = 0; u < BATCH; ++u)
#pragma unroll
      for (int it = 0; it < ITER; ++it)
        q[u][it] = (s0 + u < n_partials && kk[it] < k_end)
                       ? __ldcg(reinterpret_cast<const float4*>(P + (s0 + u) * partial_stride + (size_t)row * d + kk[it]))
                       : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int u = 0; u < BATCH; ++u)
#pragma unroll
      for (int it = 0; it < ITER; ++it) {
        v[it].x += q[u][it].x; v[it].y += q[u][it].y; v[it].z += q[u][it].z; v[it].w += q[u][it].w;
      }
  }
  if (late_status != 0) return;              // same for the whole cluster; nothing has been written yet
  float ss = 0.f;
#pragma unroll
  for (int it = 0; it < ITER; ++it) {
    if (n_partials > 0 && kk[it] < k_end) *reinterpret_cast<float4*>(x + kk[it]) = v[it];
    ss += v[it].x * v[it].x + v[it].y * v[it].y + v[it].z * v[it].z + v[it].w * v[it].w;
  }
  ss = block_sum_256(ss);
  // every CTA hands its sum to all four (slot = its rank) before the one cluster barrier; afterwards each reads
  // only its own shared memory, so nobody has to wait for a peer before leaving
  if (tid < kNormCluster) *cluster.map_shared_rank(&s_ss[rank], tid) = ss;
  cluster.sync();
  float total = 0.f;
#pragma unroll
  for (int r = 0; r < kNormCluster; ++r) total += s_ss[r];
  const float inv = rsqrtf(total / (float)d + eps);
#pragma unroll
  for (int it = 0; it < ITER; ++it) {
    if (kk[it] < k_end) {
      uint32_t ph[2], pl[2];
      split2_pack(v[it].x * inv * g[it].x, v[it].y * inv * g[it].y, ph[0], pl[0]);
      split2_pack(v[it].z * inv * g[it].z, v[it].w * inv * g[it].w, ph[1], pl[1]);
      *reinterpret_cast<uint2*>(hi + kk[it]) = make_uint2(ph[0], ph[1]);
      *reinterpret_cast<uint2*>(lo + kk[it]) = make_uint2(pl[0], pl[1]);
    }
  }
}

void launch_rmsnorm_split(specasr_kv* kv, const int32_t* ctl, const float* gain, int n, int n_pad, int n_partials,
                          cudaStream_t s) {
  const specasr_model* m = kv->m;
  const int d = m->cfg.d_model;
  const int d_part = (d + 4 * kNormCluster - 1) / (4 * kNormCluster) * 4;      // columns per CTA, a multiple of 4
  const size_t stride = (size_t)kv->n_alloc * d;
  LaunchScope scope(kv, SPECASR_KIND_NORM, s);
#define NORM_LAUNCH(I)                                                                                           \
  launch_pdl_cluster(k_rmsnorm_split<I>, dim3(kNormCluster * n_pad), dim3(256), kNormCluster, s, ctl,          \
                     kv->ws.X, kv->ws.P, n_partials, stride, gain, d, d_part, m->cfg.rms_eps, n, stride, kv->ws.H \
                     SPECASR_TRACE_ARG(kv))
  if (d_part <= 1024) NORM_LAUNCH(1);
  else if (d_part <= 2048) NORM_LAUNCH(2);
  else if (d_part <= 4096) NORM_LAUNCH(4);
  else NORM_LAUNCH(8);
#undef NORM_LAUNCH
}

// ------------------------------------------------------------------------------------------------
// Rotary embedding at tree positions + KV append.  One thread per (node, head of the fused QKV row, four
// adjacent rotation pairs).  Sums the QKV projection's partial planes (their columns follow the rotary-paired
// row order of Wqkv, in which four adjacent features are four adjacent columns), rotates Q and K heads by the
// angle of the node's position (rotate-half pairing, table built in fp64 on the host), writes Q as hi/lo planes
// and K,V as hi/lo planes into cache slot L + node.
// The grid is kept small (a few hundred blocks) on purpose: launched with programmatic stream serialization the
// blocks become resident while the QKV projection still runs, and only a grid that fits beside it in one wave
// starts working the moment the projection ends.
__global__ void __launch_bounds__(128) k_rope_append(const __grid_constant__ SegTable tab, const float* __restrict__ P,
                                                     int n_partials, size_t partial_stride, int qkv_dim, int Hq, int Hkv,
                                                     int dh, const int32_t* __restrict__ pos,
                                                     const float2* __restrict__ rope, int layer, bf16* __restrict__ Q,
                                                     size_t q_plane_stride, int page_size, int max_positions
                                                     SPECASR_TRACE_PARAM) {
  grid_dep_launch();
  SPECASR_TRACE_SCOPE(tr, SPECASR_KIND_ROPE);
  grid_dep_wait();
  SPECASR_TRACE_MARK();
  const int i = blockIdx.x;                    // workspace row
  const SegDev& sg = tab.seg[segment_of_row(tab, i)];
  const int32_t* ctl = sg.ctl;
  const int half = dh >> 1;
  const int per_head = half >> 2;              // threads per head: four rotation pairs each
  const int head = blockIdx.y * (blockDim.x / per_head) + threadIdx.x / per_head;
  const int k = (threadIdx.x % per_head) * 4;
  if (head >= Hq + 2 * Hkv) return;
  const size_t col = (size_t)i * qkv_dim + (size_t)head * dh;
  const size_t c1 = col + qkv_row_of_feature(k, dh), c2 = col + qkv_row_of_feature(k + half, dh);
  const bool is_v = head >= Hq + Hkv;
  float4 x1 = make_float4(0.f, 0.f, 0.f, 0.f), x2 = x1;
  float4 cs01 = make_float4(1.f, 0.f, 1.f, 0.f), cs23 = cs01;      // (cos, sin) of pairs k, k+1 and k+2, k+3
  int status = 0, len = 0;
  for (int s0 = 0; s0 < n_partials; s0 += 4) {   // four planes in flight, summed in plane order
    float4 a1[4], a2[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const bool on = s0 + s < n_partials;
      a1[s] = on ? __ldcg(reinterpret_cast<const float4*>(P + (s0 + s) * partial_stride + c1)) : make_float4(0.f, 0.f, 0.f, 0.f);
      a2[s] = on ? __ldcg(reinterpret_cast<const float4*>(P + (s0 + s) * partial_stride + c2)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (s0 == 0) {
      // the small loads that depend on one another (status, position -> table row, length) go out behind the
      // plane loads instead of in front of them: an in-order core would otherwise wait for each before the next
      status = ctl[CTL_STATUS];
      len = ctl[CTL_LEN];
      if (!is_v) {
        // the position is read before the status is known (a refused call never wrote it): keep the row inside the table
        const int pp = min(max(pos[i], 0), max_positions - 1);
        const float4* t = reinterpret_cast<const float4*>(rope + (size_t)pp * half + k);
        cs01 = t[0];
        cs23 = t[1];
      }
    }
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      x1.x += a1[s].x; x1.y += a1[s].y; x1.z += a1[s].z; x1.w += a1[s].w;
      x2.x += a2[s].x; x2.y += a2[s].y; x2.z += a2[s].z; x2.w += a2[s].w;
    }
  }
  if (n_partials <= 0) {
    status = ctl[CTL_STATUS];
    len = ctl[CTL_LEN];
  }
  if (status != 0) return;                       // nothing is written for an utterance whose tree was refused
  // r1 = x1 cos - x2 sin, r2 = x2 cos + x1 sin (identity for V: cos = 1, sin = 0)
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
  if (head < Hq) {
    dst = Q + (size_t)i * Hq * dh + (size_t)head * dh;
    plane = q_plane_stride;
  } else {
    const int kvh = is_v ? head - Hq - Hkv : head - Hq;
    const int slot = len + (i - sg.row0);
    const int page = sg.page_table[slot / page_size];
    const int off = slot % page_size;
    dst = (is_v ? sg.v_pool : sg.k_pool) + kv_plane_offset(layer, sg.n_pages, Hkv, page_size, dh, page, kvh, 0) +
          (size_t)off * dh;
    plane = (size_t)page_size * dh;
  }
  *reinterpret_cast<uint2*>(dst + k) = make_uint2(h1[0], h1[1]);
  *reinterpret_cast<uint2*>(dst + k + half) = make_uint2(h2[0], h2[1]);
  *reinterpret_cast<uint2*>(dst + plane + k) = make_uint2(l1[0], l1[1]);
  *reinterpret_cast<uint2*>(dst + plane + k + half) = make_uint2(l2[0], l2[1]);
}

void launch_rope_append(specasr_kv* wk, const SegTable& t, int n_total, int layer, int n_partials, cudaStream_t s) {
  const specasr_model* m = wk->m;
  const specasr_model_config& c = m->cfg;
  const int heads_per_block = 128 / (c.head_dim / 8);
  dim3 grid(n_total, (c.n_heads + 2 * c.n_kv_heads + heads_per_block - 1) / heads_per_block);
  LaunchScope scope(wk, SPECASR_KIND_ROPE, s);
  launch_pdl(k_rope_append, grid, dim3(128), 0, s, t, wk->ws.P, n_partials, (size_t)wk->n_alloc * m->qkv_dim, m->qkv_dim,
             c.n_heads, c.n_kv_heads, c.head_dim, wk->ws.pos, m->rope_table, layer, wk->ws.Q,
             (size_t)wk->n_alloc * m->q_dim, c.page_size, c.max_positions SPECASR_TRACE_ARG(wk));
}

// ------------------------------------------------------------------------------------------------
// Merge of the attention kernel's KV splits (log-sum-exp combination in base 2), normalisation and
// hi/lo split of the result for the O projection.  One warp per (node, head) row: lane s holds the
// (max, sum) of splits s and s + 32, lane c the output columns 4c .. 4c + 3; the partial outputs of
// six splits are requested together (more would cost the registers that let the blocks wait beside the attention
// kernel in one wave).  Rows n..n_pad-1 are zeroed.
__global__ void __launch_bounds__(128) k_attn_merge(const int32_t* __restrict__ ctl, const float* __restrict__ attO,
                                                    const float2* __restrict__ attML, int n_splits, size_t rows_alloc,
                                                    int Hq, int dh, int n, int rows_total, bf16* __restrict__ AO,
                                                    size_t plane_stride SPECASR_TRACE_PARAM) {
  grid_dep_launch();
  SPECASR_TRACE_SCOPE(tr, SPECASR_KIND_ATTN_MERGE);
  grid_dep_wait();
  SPECASR_TRACE_MARK();
  if (ctl[CTL_STATUS] != 0) return;
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * 4 + (threadIdx.x >> 5);       // = node * Hq + head
  if (row >= rows_total) return;
  const int c = lane * 4;
  bf16* out = AO + (size_t)row * dh + c;
  if (row / Hq >= n) {
    if (c < dh) {
      *reinterpret_cast<uint2*>(out) = make_uint2(0, 0);
      *reinterpret_cast<uint2*>(out + plane_stride) = make_uint2(0, 0);
    }
    return;
  }
  const float2 none = make_float2(-INFINITY, 0.f);
  const float2 ml0 = lane < n_splits ? __ldcg(attML + (size_t)lane * rows_alloc + row) : none;
  const float2 ml1 = lane + 32 < n_splits ? __ldcg(attML + (size_t)(lane + 32) * rows_alloc + row) : none;
  // The partial outputs are requested whatever their weights turn out to be, the first six right behind the
  // (max, sum) pairs, so that no load waits for another; an empty key block's output was never written and is
  // dropped below.
  constexpr int B6 = 6;
  float4 o[B6];
#pragma unroll
  for (int u = 0; u < B6; ++u)
    o[u] = (u < n_splits && c < dh) ? __ldcg(reinterpret_cast<const float4*>(attO + ((size_t)u * rows_alloc + row) * dh + c))
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
  float mx = fmaxf(ml0.y > 0.f ? ml0.x : -INFINITY, ml1.y > 0.f ? ml1.x : -INFINITY);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
  const float w0 = ml0.y > 0.f ? exp2f(ml0.x - mx) : 0.f;
  const float w1 = ml1.y > 0.f ? exp2f(ml1.x - mx) : 0.f;
  // denominator: the terms are added one by one in split order, so the result does not depend on timing
  float den = 0.f;
  for (int s = 0; s < n_splits; ++s) den += __shfl_sync(0xFFFFFFFFu, s < 32 ? ml0.y * w0 : ml1.y * w1, s & 31);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s0 = 0; s0 < n_splits; s0 += B6) {
    if (s0 > 0) {
#pragma unroll
      for (int u = 0; u < B6; ++u) {
        const int s = s0 + u;
        o[u] = (s < n_splits && c < dh) ? __ldcg(reinterpret_cast<const float4*>(attO + ((size_t)s * rows_alloc + row) * dh + c))
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
#pragma unroll
    for (int u = 0; u < B6; ++u) {
      const int s = s0 + u;
      float w = __shfl_sync(0xFFFFFFFFu, s < 32 ? w0 : w1, s & 31);
      if (s >= n_splits || !(w > 0.f)) {
        w = 0.f;
        o[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
      acc.x += o[u].x * w; acc.y += o[u].y * w; acc.z += o[u].z * w; acc.w += o[u].w * w;
    }
  }
  if (c < dh) {
    const float r = 1.f / den;
    uint32_t ph[2], pl[2];
    split2_pack(acc.x * r, acc.y * r, ph[0], pl[0]);
    split2_pack(acc.z * r, acc.w * r, ph[1], pl[1]);
    *reinterpret_cast<uint2*>(out) = make_uint2(ph[0], ph[1]);
    *reinterpret_cast<uint2*>(out + plane_stride) = make_uint2(pl[0], pl[1]);
  }
}

void launch_attn_merge(specasr_kv* kv, const int32_t* ctl, int n, int n_pad, int n_splits, cudaStream_t s) {
  const specasr_model_config& c = kv->m->cfg;
  const int rows_total = n_pad * c.n_heads;
  LaunchScope scope(kv, SPECASR_KIND_ATTN_MERGE, s);
  launch_pdl(k_attn_merge, dim3((rows_total + 3) / 4), dim3(128), 0, s, ctl, kv->ws.attO, kv->ws.attML, n_splits,
             (size_t)kv->n_alloc * c.n_heads, c.n_heads, c.head_dim, n, rows_total, kv->ws.AO,
             (size_t)kv->n_alloc * kv->m->q_dim SPECASR_TRACE_ARG(kv));
}

// ------------------------------------------------------------------------------------------------
// Accept: reduce the per-vocab-tile argmax candidates, then follow draft tokens while they equal the
// target's greedy token at their parent; the deepest such node (lowest index among equals) wins.
// One block per utterance; arrays indexed by workspace row, out_accept_len / out_bonus by utterance.
__global__ void __launch_bounds__(1024) k_accept(const __grid_constant__ SegTable tab, const int32_t* __restrict__ ctl_shared,
                                                const unsigned long long* __restrict__ amax, int n_tiles,
                                                int n_alloc, const int32_t* __restrict__ tokens,
                                                const int32_t* __restrict__ parent,
                                                const int32_t* __restrict__ depth,
                                                int32_t* __restrict__ out_argmax, int32_t* __restrict__ out_accept_len,
                                                int32_t* __restrict__ out_path, int32_t* __restrict__ out_bonus
                                                SPECASR_TRACE_PARAM) {
  __shared__ int s_arg[SPECASR_MAX_NODES];
  __shared__ int s_parent[SPECASR_MAX_NODES], s_token[SPECASR_MAX_NODES];   // the walks below would otherwise be
  __shared__ unsigned int s_best;                                           // chains of dependent global loads
  __shared__ unsigned long long s_red[16][64];
  SPECASR_TRACE_SCOPE(tr, SPECASR_KIND_ACCEPT);
  const int i = threadIdx.x;
  const SegDev& sg = tab.seg[blockIdx.x];
  int32_t* ctl = sg.ctl;
  const int n = sg.n;
  amax += sg.row0;
  tokens += sg.row0;
  parent += sg.row0;
  depth += sg.row0;
  out_argmax += sg.row0;
  out_path += sg.row0;
  out_accept_len += blockIdx.x;
  if (out_bonus) out_bonus += blockIdx.x;
  grid_dep_launch();
  grid_dep_wait();
  SPECASR_TRACE_MARK();
  // a failure of the kernels shared by a whole batch (a bounded wait that ran out) fails every utterance
  const int shared_status = ctl_shared ? ctl_shared[CTL_STATUS] : 0;
  if (ctl[CTL_STATUS] != 0 || shared_status != 0) {
    if (i == 0 && ctl[CTL_STATUS] == 0) ctl[CTL_STATUS] = shared_status;
    if (i < n) {
      out_path[i] = -1;
      out_argmax[i] = -1;
    }
    if (i == 0) {
      out_accept_len[0] = -1;
      if (out_bonus) out_bonus[0] = -1;
    }
    return;
  }
  if (i == 0) s_best = 0u;
  if (i < n) {
    s_parent[i] = parent[i];
    s_token[i] = tokens[i];
  }
  // arg-max over the vocabulary tiles, 64 nodes at a time: thread (node, g) scans tiles g, g + 16, ... so that a warp
  // reads 32 adjacent nodes of one tile (the candidates are [tile][node]); the 16 partial results meet in shared
  // memory.  (One warp per node with the lanes striding over the tiles touched every 32-byte sector four times and
  // took 12 us on the single SM this kernel runs on.)
  for (int node0 = 0; node0 < n; node0 += 64) {
    const int node = node0 + (i & 63), g = i >> 6;
    unsigned long long best = 0ull;
    if (node < n) {
      for (int t0 = g; t0 < n_tiles; t0 += 16 * 8) {
        unsigned long long v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int t = t0 + u * 16;
          v[u] = t < n_tiles ? __ldcg(amax + (size_t)t * n_alloc + node) : 0ull;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) best = v[u] > best ? v[u] : best;
      }
    }
    s_red[g][i & 63] = best;
    __syncthreads();
    if (i < 64 && node < n) {
#pragma unroll
      for (int q = 0; q < 16; ++q) best = s_red[q][i] > best ? s_red[q][i] : best;
      const int tok = (int)(0xFFFFFFFFu - (unsigned int)(best & 0xFFFFFFFFull));
      s_arg[node] = tok;
      out_argmax[node] = tok;
      out_path[node] = -1;
    }
    __syncthreads();
  }
  __syncthreads();
  if (i < n) {
    bool ok = true;
    int j = i;
    int steps = 0;
    while (j > 0 && steps <= n) {
      const int p = s_parent[j];
      ok = ok && (s_token[j] == s_arg[p]);
      j = p;
      ++steps;
    }
    if (ok) atomicMax(&s_best, ((unsigned int)depth[i] << 16) | (unsigned int)(0xFFFF - i));
  }
  __syncthreads();
  if (i == 0) {
    const int best = 0xFFFF - (int)(s_best & 0xFFFFu);
    const int a = (int)(s_best >> 16);
    out_accept_len[0] = a;
    if (out_bonus) out_bonus[0] = s_arg[best];
    int j = best;
    for (int k = a; k >= 0 && j >= 0; --k) {
      out_path[k] = j;
      j = s_parent[j];
    }
  }
}

void launch_accept(specasr_kv* wk, const SegTable& t, const int32_t* ctl_shared, const int32_t* tokens,
                   const int32_t* parent, int n_tiles, int32_t* out_argmax, int32_t* out_accept_len, int32_t* out_path,
                   int32_t* out_bonus, cudaStream_t s) {
  LaunchScope scope(wk, SPECASR_KIND_ACCEPT, s);
  launch_pdl(k_accept, dim3(t.count), dim3(1024), 0, s, t, ctl_shared, wk->ws.amax, n_tiles, wk->n_alloc, tokens, parent,
             wk->ws.depth, out_argmax, out_accept_len, out_path, out_bonus SPECASR_TRACE_ARG(wk));
}

// ------------------------------------------------------------------------------------------------
// Cache length bookkeeping.
__global__ void k_advance_len(int32_t* ctl, int n) {
  grid_dep_launch();
  grid_dep_wait();
  if (ctl[CTL_STATUS] != 0) return;
  ctl[CTL_LEN] += n;
}
__global__ void k_set_len(int32_t* ctl, int len) {
  grid_dep_launch();
  grid_dep_wait();
  ctl[CTL_LEN] = len;
  ctl[CTL_STATUS] = 0;
  ctl[CTL_N] = 0;
}
void launch_advance_len(specasr_kv* kv, int n, cudaStream_t s) {
  LaunchScope scope(kv, SPECASR_KIND_COMMIT, s);
  launch_pdl(k_advance_len, dim3(1), dim3(1), 0, s, kv->ws.ctl, n);
}
void launch_set_len(specasr_kv* kv, int len, cudaStream_t s) {
  LaunchScope scope(kv, SPECASR_KIND_COMMIT, s);
  launch_pdl(k_set_len, dim3(1), dim3(1), 0, s, kv->ws.ctl, len);
}

// ------------------------------------------------------------------------------------------------
// Commit: slot L+j <- slot L+path[j], j ascending.  path[j] >= j and strictly increasing, so a
// destination is never the source of a later move; each thread owns one 16-byte column of one
// (layer, pool, kv head, plane) and walks j in order, which makes the in-place copy safe.
__global__ void __launch_bounds__(256) k_commit(const int32_t* __restrict__ ctl, const int32_t* __restrict__ path,
                                                const int32_t* __restrict__ accept_len, bf16* __restrict__ k_pool,
                                                bf16* __restrict__ v_pool, const int32_t* __restrict__ page_table,
                                                int n_pages, int Hkv, int page_size, int dh) {
  grid_dep_launch();
  grid_dep_wait();
  __shared__ int s_path[SPECASR_MAX_NODES];      // read once, side by side, instead of one dependent load per step
  const int a = accept_len[0];
  const int n = ctl[CTL_N];
  if (ctl[CTL_STATUS] != 0 || a < 0 || a >= n) return;
  for (int j = threadIdx.x; j <= a; j += blockDim.x) s_path[j] = path[j];
  __syncthreads();
  const int L = ctl[CTL_LEN];
  const int layer = blockIdx.x;
  bf16* pool = blockIdx.y == 0 ? k_pool : v_pool;
  const int chunks_per_row = dh / 8;
  const int cols = Hkv * 2 * chunks_per_row;
  for (int c = threadIdx.x; c < cols; c += blockDim.x) {
    const int kvh = c / (2 * chunks_per_row);
    const int plane = (c / chunks_per_row) & 1;
    const int ch = c % chunks_per_row;
    int prev = 0;
    for (int j = 1; j <= a; ++j) {
      const int pj = s_path[j];
      if (pj <= prev || pj >= n) break;   // not a root path of the pending tree: stop copying
      prev = pj;
      if (pj == j) continue;
      const int src = L + pj, dst = L + j;
      const bf16* sp = pool + kv_plane_offset(layer, n_pages, Hkv, page_size, dh, page_table[src / page_size], kvh, plane) +
                       (size_t)(src % page_size) * dh + ch * 8;
      bf16* dp = pool + kv_plane_offset(layer, n_pages, Hkv, page_size, dh, page_table[dst / page_size], kvh, plane) +
                 (size_t)(dst % page_size) * dh + ch * 8;
      *reinterpret_cast<uint4*>(dp) = *reinterpret_cast<const uint4*>(sp);
    }
  }
}

__global__ void k_commit_finish(int32_t* ctl, const int32_t* __restrict__ accept_len) {
  grid_dep_launch();
  grid_dep_wait();
  const int a = accept_len[0];
  const int n = ctl[CTL_N];
  if (ctl[CTL_STATUS] != 0 || a < 0 || a >= n) return;
  ctl[CTL_LEN] += a + 1;
  ctl[CTL_N] = 0;
}

void launch_commit(specasr_kv* kv, const int32_t* path, const int32_t* accept_len, cudaStream_t s) {
  const specasr_model_config& c = kv->m->cfg;
  dim3 grid(c.n_layers, 2);
  LaunchScope scope(kv, SPECASR_KIND_COMMIT, s);
  launch_pdl(k_commit, grid, dim3(256), 0, s, kv->ws.ctl, path, accept_len, kv->k_pool, kv->v_pool, kv->page_table, kv->n_pages,
                                c.n_kv_heads, c.page_size, c.head_dim);
  launch_pdl(k_commit_finish, dim3(1), dim3(1), 0, s, kv->ws.ctl, accept_len);
  kv->launches++;
}
