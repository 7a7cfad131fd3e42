// Tree-masked grouped-query attention on the 5th-generation tensor cores (sm_100a).
//
// Node i sees every committed cache position [0, L) and the tree slots L + j for which j is i or an
// ancestor of i (bit j of the node's ancestor mask): the 2-D mask of a draft token tree.
//
// One CTA owns one KV head, a tile of up to 128 query rows (row = node * group + head-in-group, so a
// whole query group shares every K/V element that is staged) and one block of up to 208 cache positions,
// sized by the host so that the whole launch is one wave of CTAs:
//   S = Q K^T      M = 128 rows, N = keys, K = head_dim        (both operands K-major)
//   P = exp2(S * scale - rowmax), masked                         (two threads per row, fp32, from TMEM)
//   O = P V        M = 128 rows, N = head_dim, K = keys          (V is the MN-major B operand)
// Q, P, K and V are all carried as two bf16 planes (value ~ hi + lo); each product is three MMAs
// (hi*hi + hi*lo + lo*hi) into the same fp32 accumulator, which keeps ~16 significant bits.
// Pages of K and V arrive by TMA straight from the paged pool (one box per page, plane and 64-wide
// half of the head), Q by one box per plane and half.  Shared memory holds two regions: Q, later
// overwritten by P (in rounds of 128 keys, S stays in TMEM meanwhile), and K, later overwritten by V
// (requested as soon as the S MMAs have finished reading K), later by the output tile on its way out.
// The CTA emits an unnormalised partial (row max in log2 units, row sum, output) that k_attn_merge
// combines over the key blocks.
//
// Every mbarrier wait is bounded; on expiry the CTA records SPECASR_ERR_TIMEOUT, lets copies in
// flight land, frees its TMEM and returns.
#include "internal.h"
#include "device_utils.cuh"
#include "sm100_ptx.cuh"

using namespace sm100;

namespace {

constexpr int KEYS_MAX = 208;             // cache positions per CTA (13 pages of 16)
constexpr int ROUND = 128;                // keys whose probabilities fit the P buffer at once
constexpr int SUB = 128 * 64 * 2;         // bytes of one [128 rows][64 bf16] swizzled sub-tile (Q, P)
constexpr int KVSUB = KEYS_MAX * 64 * 2;  // bytes of one [208 keys][64 bf16] swizzled sub-tile (K, V)
constexpr int SOFTMAX_THREADS = 256;      // warps 2..9; warps w and w + 4 share a TMEM lane quadrant

struct AttnCtl {
  unsigned long long bar_qk, bar_v, bar_s, bar_p[2], bar_o[2];
  float red_max[2][128];      // per-row partial maxima / sums of the two warps that share a row
  float red_sum[2][128];
  uint32_t tmem_base;
  int abort;
};
__device__ __forceinline__ void softmax_bar() { asm volatile("bar.sync 2, 256;" ::: "memory"); }

struct AttnParams {
  int32_t* ctl;
  const int32_t* page_table;
  const unsigned long long* anc;
  float* attO;
  float2* attML;
  size_t rows_alloc;      // n_alloc * Hq
  int n_pages, page_size, layer, Hq, Hkv, group, nodes_per_tile, n, chunk, row0;
  float scale_log2;
#ifdef SPECASR_TRACE
  TraceBuf tr;
#endif
};

template <int DH>
__global__ void __launch_bounds__(64 + SOFTMAX_THREADS, 1) k_tree_attention_tc(const __grid_constant__ CUtensorMap tmQ,
                                                              const __grid_constant__ SegTable tab, AttnParams p) {
  constexpr int H = DH / 64;                               // 64-wide halves of the head
  constexpr int A_BYTES = 4 * SUB;                         // Q planes (2 H sub-tiles), later two P planes of 128 keys
  constexpr int KV_BYTES = 2 * H * KVSUB;
  extern __shared__ uint8_t smem_raw[];
  pdl_launch_dependents();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // grid z = utterance * (key blocks per utterance) + key block; the utterance's own values complete the parameters
  const int kvh = blockIdx.x, split = blockIdx.z % tab.splits;
  const SegDev& sg = tab.seg[blockIdx.z / tab.splits];
  const int node0 = blockIdx.y * p.nodes_per_tile;
  if (node0 >= sg.n) return;                               // this utterance has fewer row tiles than the largest one
  p.ctl = sg.ctl;
  p.page_table = sg.page_table;
  p.n_pages = sg.n_pages;
  p.n = sg.n;
  p.chunk = sg.chunk;
  p.row0 = sg.row0;
  p.anc += (size_t)sg.row0 * 4;
  p.attO += (size_t)sg.row0 * p.Hq * DH;
  p.attML += (size_t)sg.row0 * p.Hq;
  const CUtensorMap* tmK = sg.tmK;
  const CUtensorMap* tmV = sg.tmV;
  const int rows_used = p.nodes_per_tile * p.group;
  const int k_begin = split * p.chunk;

  uint8_t* As = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* KVs = As + A_BYTES;
  AttnCtl* sc = (AttnCtl*)(KVs + KV_BYTES);

  if (threadIdx.x == 0) {
    mbar_init(&sc->bar_qk, 1);
    mbar_init(&sc->bar_v, 1);
    mbar_init(&sc->bar_s, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sc->bar_p[i], SOFTMAX_THREADS);
      mbar_init(&sc->bar_o[i], 1);
    }
    sc->abort = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(tmK);
    tma_prefetch_desc(tmV);
  }
  if (rows_used < 128) {             // query rows the TMA box does not cover must not hold garbage
    const int chunks = (128 - rows_used) * 8;
    for (int sub = 0; sub < 2 * H; ++sub)
      for (int i = threadIdx.x; i < chunks; i += blockDim.x)
        *reinterpret_cast<uint4*>(As + sub * SUB + rows_used * 128 + i * 16) = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
  }
  if (warp == 1) tmem_alloc(&sc->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // The page table does not change during a call: lane j of the producer warp looks up the page of its key block
  // now, so that after the wait only the length stands between it and the first K load.
  int my_page = 0;
  if (warp == 0) {
    const int idx = split * (p.chunk / p.page_size) + lane;
    if (lane < p.chunk / p.page_size && idx * p.page_size < sg.capacity) my_page = p.page_table[idx];
  }
  // everything above is independent of the previous kernel; its results are read from here on
  SPECASR_TRACE_SCOPE(p.tr, SPECASR_KIND_ATTN);
  pdl_wait();
  SPECASR_TRACE_MARK();
  const bool live = p.ctl[CTL_STATUS] == 0;
  const int L = p.ctl[CTL_LEN];
  const int Ltot = L + p.n;
  // row owned by a softmax thread (warps 2..9): TMEM lane = 32 * (warp % 4) + lane
  const int r = ((warp & 3) << 5) | lane;
  const int node = node0 + r / p.group;
  const bool row_valid = warp >= 2 && r < rows_used && node < p.n;
  const size_t out_row = (size_t)split * p.rows_alloc + (size_t)node * p.Hq + kvh * p.group + r % p.group;

  const bool active = live && k_begin < Ltot;
  if (live && !active && row_valid) p.attML[out_row] = make_float2(-INFINITY, 0.f);   // key block beyond the cache: an empty partial
  const int kc = min(p.chunk, Ltot - k_begin);
  const int kc_pad = (kc + 15) & ~15;
  const int pages = (kc + p.page_size - 1) / p.page_size;
  const int rounds = (kc_pad + ROUND - 1) / ROUND;          // 1 or 2

  const uint32_t tmem_s = sc->tmem_base;           // S: columns [0, 208)
  const uint32_t tmem_o = sc->tmem_base + 256;     // O: columns [256, 256 + DH)
  volatile int* abort = &sc->abort;
  int32_t* status = p.ctl + CTL_STATUS;

  if (!active) {
    // nothing to do for this CTA
  } else if (warp == 0) {
    // ---------------- TMA producer: lane 0 fetches Q, lane j fetches page j of K and later of V
    const uint32_t q_bytes = 2 * H * rows_used * 128;
    const uint32_t kv_bytes = 2 * H * pages * p.page_size * 128;
    if (lane == 0) {
      mbar_expect_tx(&sc->bar_qk, q_bytes + kv_bytes);
      mbar_expect_tx(&sc->bar_v, kv_bytes);
    }
    __syncwarp();
    if (lane == 0) {
      for (int plane = 0; plane < 2; ++plane)
        for (int h = 0; h < H; ++h)
          tma_load_4d(As + (plane * H + h) * SUB, &tmQ, h * 64, kvh * p.group, p.row0 + node0, plane, &sc->bar_qk);
    }
    int c4 = 0;
    const int off = lane * p.page_size * 128;
    if (lane < pages) {
      c4 = p.layer * p.n_pages + my_page;
      for (int plane = 0; plane < 2; ++plane)
        for (int h = 0; h < H; ++h)
          tma_load_5d(KVs + (plane * H + h) * KVSUB + off, tmK, h * 64, 0, plane, kvh, c4, &sc->bar_qk);
    }
    // V takes K's place once the S MMAs have read K
    const bool ok = mbar_wait(&sc->bar_s, 0u, abort, status);
    if (ok && lane < pages) {
      for (int plane = 0; plane < 2; ++plane)
        for (int h = 0; h < H; ++h)
          tma_load_5d(KVs + (plane * H + h) * KVSUB + off, tmV, h * 64, 0, plane, kvh, c4, &sc->bar_v);
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer
    bool ok = mbar_wait(&sc->bar_qk, 0u, abort, status);
    if (ok) {
      tc_fence_after();
      const uint32_t idesc = make_idesc_bf16(kc_pad);
      const uint32_t a0 = smem_u32(As), b0 = smem_u32(KVs);
      uint32_t acc = 0u;
#pragma unroll
      for (int term = 0; term < 3; ++term) {
        const int qp = term == 2 ? 1 : 0, kp = term == 1 ? 1 : 0;     // hi*hi, hi*lo, lo*hi
        for (int h = 0; h < H; ++h) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            umma_bf16(tmem_s, make_smem_desc(a0 + (qp * H + h) * SUB + k * 32),
                      make_smem_desc(b0 + (kp * H + h) * KVSUB + k * 32), idesc, acc);
            acc = 1u;
          }
        }
      }
      umma_commit(&sc->bar_s);
      ok = mbar_wait(&sc->bar_v, 0u, abort, status);
    }
    const uint32_t idesc2 = make_idesc_bf16(DH, true);
    uint32_t acc = 0u;
    for (int rd = 0; rd < rounds && ok; ++rd) {
      ok = mbar_wait(&sc->bar_p[rd], 0u, abort, status);
      if (!ok) break;
      tc_fence_after();
      const uint32_t a0 = smem_u32(As), b0 = smem_u32(KVs);
      const int j_end = min(kc_pad - rd * ROUND, ROUND) / 16;
#pragma unroll
      for (int term = 0; term < 3; ++term) {
        const int pp = term == 2 ? 1 : 0, vp = term == 1 ? 1 : 0;
        for (int j = 0; j < j_end; ++j) {
          // A: P plane pp, 64-key block j / 4 of this round, 16 keys = 32 bytes along the row
          // B: V plane vp, keys of this step are rows of 128 bytes; the second half of the head is KVSUB further on
          umma_bf16(tmem_o, make_smem_desc(a0 + (pp * 2 + (j >> 2)) * SUB + (j & 3) * 32),
                    make_smem_desc(b0 + vp * H * KVSUB + (rd * (ROUND / 16) + j) * 2048, KVSUB), idesc2, acc);
          acc = 1u;
        }
      }
      umma_commit(&sc->bar_o[rd]);
    }
  } else if (warp >= 2) {
    // ---------------- softmax and epilogue: two threads per query row (warps w and w + 4), each taking
    // alternate 32-key chunks.  The chunk loops are kept rolled on purpose: straight-line code that runs
    // once is bound by instruction fetch.
    const int eg = (warp - 2) >> 2;
    unsigned long long anc0 = 0ull, anc1 = 0ull, anc2 = 0ull, anc3 = 0ull;
    if (row_valid) {
      anc0 = p.anc[node * 4 + 0];
      anc1 = p.anc[node * 4 + 1];
      anc2 = p.anc[node * 4 + 2];
      anc3 = p.anc[node * 4 + 3];
    }
    auto visible_keys = [&](int base) -> uint32_t {
      const int t0 = base - L;                      // tree slot of the chunk's first key
      if (t0 <= -32) return 0xFFFFFFFFu;            // all 32 keys lie in the committed prefix
      const int ts = t0 > 0 ? t0 : 0;
      uint32_t win = 0u;                            // ancestor bits of tree slots ts .. ts + 31
      if (ts < SPECASR_MAX_NODES) {
        const int w = ts >> 6, sh = ts & 63;
        const unsigned long long a = w == 0 ? anc0 : w == 1 ? anc1 : w == 2 ? anc2 : anc3;
        const unsigned long long b = w == 0 ? anc1 : w == 1 ? anc2 : w == 2 ? anc3 : 0ull;
        win = (uint32_t)(sh ? (a >> sh) | (b << (64 - sh)) : a);
      }
      return t0 < 0 ? ((1u << (-t0)) - 1u) | (win << (-t0)) : win;
    };
    // bit j of the result = key (k_begin + c0 + j) belongs to this CTA's block and is visible to this row
    auto visible32 = [&](int c0) -> uint32_t {
      const uint32_t mine = kc - c0 >= 32 ? 0xFFFFFFFFu : (1u << (kc - c0)) - 1u;   // c0 < kc always
      return mine & visible_keys(k_begin + c0);
    };
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    bool ok = mbar_wait(&sc->bar_s, 0u, abort, status);
    float m_row = -INFINITY;
    if (ok) {
      tc_fence_after();
      float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll 1
      for (int c0 = eg * 32; c0 < kc_pad; c0 += 64) {
        float s[32];
        tmem_ld32(tmem_s + lane_off + c0, s);
        const uint32_t vis = visible32(c0);
#pragma unroll
        for (int j = 0; j < 32; ++j) m4[j & 3] = fmaxf(m4[j & 3], ((vis >> j) & 1u) ? s[j] * p.scale_log2 : -INFINITY);
      }
      m_row = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
    }
    sc->red_max[eg][r] = m_row;
    softmax_bar();
    m_row = fmaxf(sc->red_max[0][r], sc->red_max[1][r]);
    const float m_use = m_row > -INFINITY ? m_row : 0.f;      // a fully masked row gives p = 0 everywhere
    float l2[2] = {0.f, 0.f};
    for (int rd = 0; rd < rounds && ok; ++rd) {
      // the P buffer holds 128 keys: the second round waits until the first round's MMAs have read it
      if (rd > 0) ok = mbar_wait(&sc->bar_o[rd - 1], 0u, abort, status);
      if (!ok) break;
      const int c_end = min(kc_pad, (rd + 1) * ROUND);
#pragma unroll 1
      for (int c0 = rd * ROUND + eg * 32; c0 < c_end; c0 += 64) {
        float s[32];
        tmem_ld32(tmem_s + lane_off + c0, s);
        const uint32_t vis = visible32(c0);
#pragma unroll
        for (int j = 0; j < 32; ++j) s[j] = ((vis >> j) & 1u) ? fast_exp2(s[j] * p.scale_log2 - m_use) : 0.f;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          uint32_t hi[4], lo[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int j = g * 8 + 2 * e;
            l2[e & 1] += s[j] + s[j + 1];
            split2_pack(s[j], s[j + 1], hi[e], lo[e]);
          }
          const int c8 = ((c0 - rd * ROUND) >> 3) + g;         // 8-key group within this round's 128 keys
          if (rd * ROUND + c8 * 8 < kc_pad) {
            const int off = (c8 >> 3) * SUB + r * 128 + (((c8 & 7) ^ (r & 7)) << 4);
            *reinterpret_cast<uint4*>(As + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *reinterpret_cast<uint4*>(As + 2 * SUB + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
          }
        }
      }
      if (rd == rounds - 1 && kc < kc_pad) {
        // value rows past the end of the cache meet p = 0, but 0 * garbage could still be NaN: clear them
        ok = mbar_wait(&sc->bar_v, 0u, abort, status);
        if (ok && eg == 0 && r < kc_pad - kc) {
          for (int sub = 0; sub < 2 * H; ++sub)
            for (int i = 0; i < 8; ++i)
              *reinterpret_cast<uint4*>(KVs + sub * KVSUB + (kc + r) * 128 + i * 16) = make_uint4(0, 0, 0, 0);
        }
      }
      if (ok) {
        fence_proxy_async_smem();
        mbar_arrive(&sc->bar_p[rd]);
      }
    }
    sc->red_sum[eg][r] = l2[0] + l2[1];
    if (ok) ok = mbar_wait(&sc->bar_o[rounds - 1], 0u, abort, status);
    // O leaves through the (now idle) K/V region so that a warp writes whole rows: each thread parks its part of
    // its row with the 16-byte columns rotated by the row number, then lane c reads column c of a row.
    float4* stage = reinterpret_cast<float4*>(KVs);
    constexpr int C4 = DH / 4;                               // float4 columns per row
    if (ok) {
      tc_fence_after();
#pragma unroll 1
      for (int c0 = eg * 32; c0 < DH; c0 += 64) {
        float o[32];
        tmem_ld32(tmem_o + lane_off + c0, o);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int c4 = (c0 >> 2) + e;
          stage[r * C4 + (c4 ^ (r & (C4 - 1)))] = make_float4(o[4 * e], o[4 * e + 1], o[4 * e + 2], o[4 * e + 3]);
        }
      }
    }
    softmax_bar();
    if (ok) {
      const int r_base = (warp - 2) * 16;                    // eight warps, sixteen rows each
#pragma unroll 1
      for (int i = 0; i < 16; ++i) {
        const int rr = r_base + i;
        const int nd = node0 + rr / p.group;
        if (rr < rows_used && nd < p.n) {
          const size_t orow = (size_t)split * p.rows_alloc + (size_t)nd * p.Hq + kvh * p.group + rr % p.group;
          float4* dst = reinterpret_cast<float4*>(p.attO + orow * DH);
          for (int c4 = lane; c4 < C4; c4 += 32) dst[c4] = stage[rr * C4 + (c4 ^ (rr & (C4 - 1)))];
        }
      }
      if (row_valid && eg == 0) p.attML[out_row] = make_float2(m_row, sc->red_sum[0][r] + sc->red_sum[1][r]);
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
    tmem_dealloc(sc->tmem_base, 512);
  }
}

template <int DH>
void launch_dh(specasr_kv* wk, const SegTable& t, int n_max, int layer, cudaStream_t s) {
  const specasr_model* m = wk->m;
  const specasr_model_config& c = m->cfg;
  constexpr int H = DH / 64;
  const size_t smem = 4 * SUB + 2 * H * KVSUB + sizeof(AttnCtl) + 1024;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(k_tree_attention_tc<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    configured = true;
  }
  AttnParams p;
  memset(&p, 0, sizeof(p));          // ctl, page table, n, chunk, row0, n_pages come from the utterance's table entry
  p.anc = wk->ws.anc;
  p.attO = wk->ws.attO;
  p.attML = wk->ws.attML;
  p.rows_alloc = (size_t)wk->n_alloc * c.n_heads;
  p.page_size = c.page_size;
  p.layer = layer;
  p.Hq = c.n_heads;
  p.Hkv = c.n_kv_heads;
  p.group = c.n_heads / c.n_kv_heads;
  p.nodes_per_tile = 128 / p.group;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
#ifdef SPECASR_TRACE
  p.tr = wk->trace;
#endif
  dim3 grid(c.n_kv_heads, (n_max + p.nodes_per_tile - 1) / p.nodes_per_tile, t.count * t.splits);
  LaunchScope scope(wk, SPECASR_KIND_ATTN, s);
  launch_pdl(k_tree_attention_tc<DH>, grid, dim3(64 + SOFTMAX_THREADS), smem, s, wk->tm_Q, t, p);
}

}  // namespace

bool attention_tc_supported(const specasr_model* m) {
  const specasr_model_config& c = m->cfg;
  const int group = c.n_heads / c.n_kv_heads;
  return c.gemm_path == 0 && (c.head_dim == 64 || c.head_dim == 128) && c.page_size % 16 == 0 &&
         c.page_size <= KEYS_MAX && group <= 128;
}

// Keys per CTA and number of key blocks for `total_len` positions seen by `n` nodes: as few blocks as the
// shared-memory tile allows, but enough to give each of `sm_budget` SMs a CTA.  Returns false if they exceed
// `max_splits`.
bool attention_tc_plan(const specasr_model* m, int n, int total_len, int sm_budget, int max_splits, int* n_splits,
                       int* chunk) {
  const specasr_model_config& c = m->cfg;
  const int group = c.n_heads / c.n_kv_heads;
  const int nodes_per_tile = 128 / group;
  const int ctas = c.n_kv_heads * ((n + nodes_per_tile - 1) / nodes_per_tile);
  const int keys_max = KEYS_MAX / c.page_size * c.page_size;
  int splits = (total_len + keys_max - 1) / keys_max;
  const int fill = sm_budget / ctas;                      // blocks that still fit in one wave
  if (fill > splits) splits = fill;
  if (splits > max_splits) splits = max_splits;
  // A cache that needs more key blocks than one wave holds: instead of a full second wave of 208-key blocks (of which
  // only a fraction is needed), cut it into as many blocks as whole waves can take, so that every round is shorter.
  if (splits * ctas > sm_budget && ctas <= sm_budget) {
    const int waves = (splits * ctas + sm_budget - 1) / sm_budget;
    int s2 = waves * sm_budget / ctas;
    if (s2 > max_splits) s2 = max_splits;
    if (s2 > splits) splits = s2;
  }
  int per = (total_len + splits - 1) / splits;
  per = (per + c.page_size - 1) / c.page_size * c.page_size;
  if (per < c.page_size) per = c.page_size;
  if (per > keys_max) per = keys_max;
  splits = (total_len + per - 1) / per;
  if (splits < 1) splits = 1;
  *n_splits = splits;
  *chunk = per;
  return splits <= max_splits;
}

// Tensor maps of the rotated queries and of the two pools, as the kernel above walks them.
bool attention_tc_make_maps(specasr_kv* kv) {
  const specasr_model* m = kv->m;
  const specasr_model_config& c = m->cfg;
  const int group = c.n_heads / c.n_kv_heads;
  const uint64_t dh = c.head_dim;
  {  // Q: [plane][node][head][dh]; box = 64 of dh, the `group` heads of one KV head, 128 / group nodes
    uint64_t dims[4] = {dh, (uint64_t)c.n_heads, (uint64_t)kv->n_alloc, 2};
    uint64_t strides[3] = {dh * 2, (uint64_t)m->q_dim * 2, (uint64_t)kv->n_alloc * m->q_dim * 2};
    uint32_t box[4] = {64, (uint32_t)group, (uint32_t)(128 / group), 1};
    if (!make_tensor_map_nd(&kv->tm_Q, kv->ws.Q, 4, dims, strides, box)) return false;
  }
  const uint64_t ps = c.page_size;
  uint64_t dims[5] = {dh, ps, 2, (uint64_t)c.n_kv_heads, (uint64_t)c.n_layers * kv->n_pages};
  uint64_t strides[4] = {dh * 2, ps * dh * 2, 2 * ps * dh * 2, (uint64_t)c.n_kv_heads * 2 * ps * dh * 2};
  uint32_t box[5] = {64, (uint32_t)ps, 1, 1, 1};
  if (!make_tensor_map_nd(&kv->tm_K, kv->k_pool, 5, dims, strides, box) ||
      !make_tensor_map_nd(&kv->tm_V, kv->v_pool, 5, dims, strides, box))
    return false;
  // the kernel reads the pool descriptors through the utterance table, i.e. from global memory
  cudaError_t e = cudaMemcpy(kv->ws.tmKV, &kv->tm_K, sizeof(CUtensorMap), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(kv->ws.tmKV + 1, &kv->tm_V, sizeof(CUtensorMap), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    set_error("attention descriptors: %s", cudaGetErrorString(e));
    return false;
  }
  return true;
}

void launch_tree_attention_tc(specasr_kv* wk, const SegTable& t, int n_max, int layer, cudaStream_t s) {
  if (wk->m->cfg.head_dim == 64) launch_dh<64>(wk, t, n_max, layer, s);
  else launch_dh<128>(wk, t, n_max, layer, s);
}
