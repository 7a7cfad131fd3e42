// Integer and element-wise kernels of the verification step: tree preparation, embedding gather,
// RMSNorm with operand split, rotary embedding + KV append, attention merge, accept, commit.
#include "internal.h"
#include "device_utils.cuh"

// ------------------------------------------------------------------------------------------------
// Tree preparation: validates the parent array, derives depth, position and the ancestor-or-self
// bitmask of every node (the rows of the 2-D tree attention mask), and sets the status word that
// every later kernel of the call checks.
__global__ void k_tree_prep(int32_t* __restrict__ ctl, const int32_t* __restrict__ tokens,
                            const int32_t* __restrict__ parent, int n, int vocab, int capacity,
                            int32_t* __restrict__ depth, int32_t* __restrict__ pos,
                            unsigned long long* __restrict__ anc) {
  __shared__ int s_bad;
  const int i = threadIdx.x;
  grid_dep_launch();
  grid_dep_wait();
  if (i == 0) s_bad = 0;
  __syncthreads();
  const int L = ctl[CTL_LEN];
  if (i < n) {
    const int p = parent[i];
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
      j = parent[j];
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
__global__ void k_chain_prep(int32_t* __restrict__ ctl, int n, int capacity, int32_t* __restrict__ depth,
                             int32_t* __restrict__ pos, unsigned long long* __restrict__ anc) {
  const int i = threadIdx.x;
  grid_dep_launch();
  grid_dep_wait();
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

void launch_tree_prep(specasr_kv* kv, const int32_t* tokens, const int32_t* parent, int n, cudaStream_t s) {
  const specasr_model* m = kv->m;
  int cap = kv->max_pages * m->cfg.page_size;
  if (m->cfg.max_positions < cap) cap = m->cfg.max_positions;
  LaunchScope scope(kv, SPECASR_KIND_PREP, s);
  launch_pdl(k_tree_prep, dim3(1), dim3(256), 0, s, kv->ws.ctl, tokens, parent, n, m->cfg.vocab, cap, kv->ws.depth, kv->ws.pos,
                                kv->ws.anc);
}

void launch_chain_prep(specasr_kv* kv, int n, cudaStream_t s) {
  const specasr_model* m = kv->m;
  int cap = kv->max_pages * m->cfg.page_size;
  if (m->cfg.max_positions < cap) cap = m->cfg.max_positions;
  LaunchScope scope(kv, SPECASR_KIND_PREP, s);
  launch_pdl(k_chain_prep, dim3(1), dim3(256), 0, s, kv->ws.ctl, n, cap, kv->ws.depth, kv->ws.pos, kv->ws.anc);
}

// ------------------------------------------------------------------------------------------------
// Layer-0 inputs: embedding rows (bf16 -> fp32 residual stream), or caller-provided vectors.
__global__ void k_embed_tokens(const int32_t* __restrict__ ctl, const int32_t* __restrict__ tokens,
                               const bf16* __restrict__ E, int d, float* __restrict__ X) {
  grid_dep_launch();
  grid_dep_wait();
  if (ctl[CTL_STATUS] != 0) return;
  const int i = blockIdx.x;
  const bf16* row = E + (size_t)tokens[i] * d;
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

void launch_embed_tokens(specasr_kv* kv, const int32_t* tokens, int n, cudaStream_t s) {
  LaunchScope scope(kv, SPECASR_KIND_PREP, s);
  launch_pdl(k_embed_tokens, dim3(n), dim3(128), 0, s, kv->ws.ctl, tokens, kv->m->embed, kv->m->cfg.d_model, kv->ws.X);
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
__global__ void __launch_bounds__(256) k_rmsnorm_split(const int32_t* __restrict__ ctl, float* __restrict__ X,
                                                       const float* __restrict__ P, int n_partials,
                                                       size_t partial_stride, const float* __restrict__ gain, int d, float eps, int n,
                                                       size_t plane_stride, bf16* __restrict__ H) {
  grid_dep_launch();
  grid_dep_wait();
  if (ctl[CTL_STATUS] != 0) return;
  const int row = blockIdx.x;
  bf16* hi = H + (size_t)row * d;
  bf16* lo = hi + plane_stride;
  if (row >= n) {
    for (int k = threadIdx.x * 8; k < d; k += blockDim.x * 8) {
      *reinterpret_cast<uint4*>(hi + k) = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4*>(lo + k) = make_uint4(0, 0, 0, 0);
    }
    return;
  }
  float* x = X + (size_t)row * d;
  float ss = 0.f;
  for (int k = threadIdx.x * 4; k < d; k += blockDim.x * 4) {
    float4 v = *reinterpret_cast<const float4*>(x + k);
    for (int s = 0; s < n_partials; ++s) {
      const float4 p = __ldcg(reinterpret_cast<const float4*>(P + s * partial_stride + (size_t)row * d + k));
      v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
    }
    if (n_partials > 0) *reinterpret_cast<float4*>(x + k) = v;
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = block_sum_256(ss);
  const float inv = rsqrtf(ss / (float)d + eps);
  for (int k = threadIdx.x * 4; k < d; k += blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4*>(x + k);
    const float4 g = *reinterpret_cast<const float4*>(gain + k);
    const float h[4] = {v.x * inv * g.x, v.y * inv * g.y, v.z * inv * g.z, v.w * inv * g.w};
    uint32_t ph[2], pl[2];
    split2_pack(h[0], h[1], ph[0], pl[0]);
    split2_pack(h[2], h[3], ph[1], pl[1]);
    *reinterpret_cast<uint2*>(hi + k) = make_uint2(ph[0], ph[1]);
    *reinterpret_cast<uint2*>(lo + k) = make_uint2(pl[0], pl[1]);
  }
}

void launch_rmsnorm_split(specasr_kv* kv, const float* gain, int n, int n_pad, int n_partials, cudaStream_t s) {
  const specasr_model* m = kv->m;
  const int d = m->cfg.d_model;
  LaunchScope scope(kv, SPECASR_KIND_NORM, s);
  launch_pdl(k_rmsnorm_split, dim3(n_pad), dim3(256), 0, s, kv->ws.ctl, kv->ws.X, kv->ws.P, n_partials, (size_t)kv->n_alloc * d, gain,
             d, m->cfg.rms_eps, n, (size_t)kv->n_alloc * d, kv->ws.H);
}

// ------------------------------------------------------------------------------------------------
// Rotary embedding at tree positions + KV append.  One block per (node, head of the fused QKV row).
// Sums the QKV projection's partial planes (their columns follow the rotary-paired row order of Wqkv),
// rotates Q and K heads by the angle of
// the node's position (rotate-half pairing, table built in fp64 on the host), writes Q as hi/lo planes
// and K,V as hi/lo planes into cache slot L + node.
__global__ void k_rope_append(const int32_t* __restrict__ ctl, const float* __restrict__ P, int n_partials,
                              size_t partial_stride, int qkv_dim, int Hq, int Hkv, int dh, const int32_t* __restrict__ pos, const float2* __restrict__ rope,
                              int layer, bf16* __restrict__ Q, size_t q_plane_stride, bf16* __restrict__ k_pool,
                              bf16* __restrict__ v_pool, const int32_t* __restrict__ page_table, int n_pages,
                              int page_size) {
  grid_dep_launch();
  grid_dep_wait();
  if (ctl[CTL_STATUS] != 0) return;
  const int i = blockIdx.x;
  const int head = blockIdx.y;
  const int half = dh >> 1;
  const int k = threadIdx.x;
  if (k >= half) return;
  const size_t col = (size_t)i * qkv_dim + (size_t)head * dh;
  const size_t c1 = col + qkv_row_of_feature(k, dh), c2 = col + qkv_row_of_feature(k + half, dh);
  float x1 = 0.f, x2 = 0.f;
  for (int s = 0; s < n_partials; ++s) {
    x1 += __ldcg(P + s * partial_stride + c1);
    x2 += __ldcg(P + s * partial_stride + c2);
  }
  const bool is_v = head >= Hq + Hkv;
  if (!is_v) {
    const float2 cs = rope[(size_t)pos[i] * half + k];
    const float r1 = x1 * cs.x - x2 * cs.y;
    const float r2 = x2 * cs.x + x1 * cs.y;
    x1 = r1;
    x2 = r2;
  }
  bf16 h1, l1, h2, l2;
  split_bf16(x1, h1, l1);
  split_bf16(x2, h2, l2);
  if (head < Hq) {
    bf16* q = Q + (size_t)i * Hq * dh + (size_t)head * dh;
    q[k] = h1;
    q[k + half] = h2;
    q[q_plane_stride + k] = l1;
    q[q_plane_stride + k + half] = l2;
  } else {
    const int kvh = is_v ? head - Hq - Hkv : head - Hq;
    const int slot = ctl[CTL_LEN] + i;
    const int page = page_table[slot / page_size];
    const int off = slot % page_size;
    bf16* pool = is_v ? v_pool : k_pool;
    bf16* dst = pool + kv_plane_offset(layer, n_pages, Hkv, page_size, dh, page, kvh, 0) + (size_t)off * dh;
    const size_t plane = (size_t)page_size * dh;
    dst[k] = h1;
    dst[k + half] = h2;
    dst[plane + k] = l1;
    dst[plane + k + half] = l2;
  }
}

void launch_rope_append(specasr_kv* kv, int layer, int n, int n_partials, cudaStream_t s) {
  const specasr_model* m = kv->m;
  const specasr_model_config& c = m->cfg;
  dim3 grid(n, c.n_heads + 2 * c.n_kv_heads);
  const int threads = c.head_dim / 2 < 32 ? 32 : c.head_dim / 2;
  LaunchScope scope(kv, SPECASR_KIND_ROPE, s);
  launch_pdl(k_rope_append, grid, dim3(threads), 0, s, kv->ws.ctl, kv->ws.P, n_partials, (size_t)kv->n_alloc * m->qkv_dim, m->qkv_dim, c.n_heads, c.n_kv_heads,
             c.head_dim, kv->ws.pos, m->rope_table, layer, kv->ws.Q, (size_t)kv->n_alloc * m->q_dim, kv->k_pool,
             kv->v_pool, kv->page_table, kv->n_pages, c.page_size);
}

// ------------------------------------------------------------------------------------------------
// Merge of the attention kernel's KV splits (log-sum-exp combination in base 2), normalisation and
// hi/lo split of the result for the O projection.  Rows n..n_pad-1 are zeroed.
__global__ void k_attn_merge(const int32_t* __restrict__ ctl, const float* __restrict__ attO,
                             const float2* __restrict__ attML, int n_splits, size_t rows_alloc, int Hq, int dh,
                             int n, bf16* __restrict__ AO, size_t plane_stride) {
  grid_dep_launch();
  grid_dep_wait();
  if (ctl[CTL_STATUS] != 0) return;
  const int i = blockIdx.x;
  const int h = blockIdx.y;
  const int d = threadIdx.x;
  if (d >= dh) return;
  bf16* out = AO + (size_t)i * Hq * dh + (size_t)h * dh + d;
  if (i >= n) {
    out[0] = __float2bfloat16_rn(0.f);
    out[plane_stride] = __float2bfloat16_rn(0.f);
    return;
  }
  const size_t row = (size_t)i * Hq + h;
  float mx = -INFINITY;
  for (int s = 0; s < n_splits; ++s) mx = fmaxf(mx, attML[s * rows_alloc + row].x);
  float num = 0.f, den = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    const float2 ml = attML[s * rows_alloc + row];
    if (ml.y > 0.f) {
      const float w = exp2f(ml.x - mx);
      den += ml.y * w;
      num += attO[(s * rows_alloc + row) * dh + d] * w;
    }
  }
  const float o = num / den;
  bf16 hi, lo;
  split_bf16(o, hi, lo);
  out[0] = hi;
  out[plane_stride] = lo;
}

void launch_attn_merge(specasr_kv* kv, int n, int n_pad, int n_splits, cudaStream_t s) {
  const specasr_model_config& c = kv->m->cfg;
  dim3 grid(n_pad, c.n_heads);
  const int threads = c.head_dim < 32 ? 32 : c.head_dim;
  LaunchScope scope(kv, SPECASR_KIND_ATTN_MERGE, s);
  launch_pdl(k_attn_merge, grid, dim3(threads), 0, s, kv->ws.ctl, kv->ws.attO, kv->ws.attML, n_splits,
                                        (size_t)kv->n_alloc * c.n_heads, c.n_heads, c.head_dim, n, kv->ws.AO,
                                        (size_t)kv->n_alloc * kv->m->q_dim);
}

// ------------------------------------------------------------------------------------------------
// Accept: reduce the per-vocab-tile argmax candidates, then follow draft tokens while they equal the
// target's greedy token at their parent; the deepest such node (lowest index among equals) wins.
__global__ void __launch_bounds__(256) k_accept(const int32_t* __restrict__ ctl,
                                                const unsigned long long* __restrict__ amax, int n_tiles,
                                                int n_alloc, const int32_t* __restrict__ tokens,
                                                const int32_t* __restrict__ parent,
                                                const int32_t* __restrict__ depth, int n,
                                                int32_t* __restrict__ out_argmax, int32_t* __restrict__ out_accept_len,
                                                int32_t* __restrict__ out_path, int32_t* __restrict__ out_bonus) {
  __shared__ int s_arg[SPECASR_MAX_NODES];
  __shared__ unsigned int s_best;
  const int i = threadIdx.x;
  grid_dep_launch();
  grid_dep_wait();
  if (ctl[CTL_STATUS] != 0) {
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
    unsigned long long best = 0ull;
    for (int t = 0; t < n_tiles; ++t) {
      const unsigned long long v = amax[(size_t)t * n_alloc + i];
      best = v > best ? v : best;
    }
    const int tok = (int)(0xFFFFFFFFu - (unsigned int)(best & 0xFFFFFFFFull));
    s_arg[i] = tok;
    out_argmax[i] = tok;
    out_path[i] = -1;
  }
  __syncthreads();
  if (i < n) {
    bool ok = true;
    int j = i;
    int steps = 0;
    while (j > 0 && steps <= n) {
      const int p = parent[j];
      ok = ok && (tokens[j] == s_arg[p]);
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
      j = parent[j];
    }
  }
}

void launch_accept(specasr_kv* kv, const int32_t* tokens, const int32_t* parent, int n, int n_tiles,
                   int32_t* out_argmax, int32_t* out_accept_len, int32_t* out_path, int32_t* out_bonus,
                   cudaStream_t s) {
  LaunchScope scope(kv, SPECASR_KIND_ACCEPT, s);
  launch_pdl(k_accept, dim3(1), dim3(256), 0, s, kv->ws.ctl, kv->ws.amax, n_tiles, kv->n_alloc, tokens, parent, kv->ws.depth, n,
                             out_argmax, out_accept_len, out_path, out_bonus);
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
  const int a = accept_len[0];
  const int n = ctl[CTL_N];
  if (ctl[CTL_STATUS] != 0 || a < 0 || a >= n) return;
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
      const int pj = path[j];
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
