// C ABI entry points: handle management, host-side validation and the kernel sequence of one
// verification round.  See include/specasr.h for the contract of every call.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "internal.h"
#include "device_utils.cuh"

// ------------------------------------------------------------------------------------------------
static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

extern "C" const char* specasr_last_error(void) { return g_err; }

#define CUDA_TRY(expr)                                                              \
  do {                                                                              \
    cudaError_t e__ = (expr);                                                       \
    if (e__ != cudaSuccess) {                                                       \
      set_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__), __FILE__, __LINE__); \
      return SPECASR_ERR_CUDA;                                                      \
    }                                                                               \
  } while (0)

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
// Token counts are padded to 16, 32, 64, 128 or 256 so that the activation block of a projection is one TMA box
// and one MMA (a padded count like 48 would need three narrow MMAs per k-step).
static inline int pad_tokens(int n) {
  int p = 16;
  while (p < n) p <<= 1;
  return p;
}

// The plain-FMA projections and the plain attention kernel are a second engine kept for cross-checking kernels on a
// GPU.  They are compiled only into the library variant built with -DSPECASR_CROSSCHECK; the product library has the
// tensor-core path alone and refuses what that path does not cover.
int lm_tiles_of(const specasr_model* m) {
#ifdef SPECASR_CROSSCHECK
  if (m->cfg.gemm_path == 1) return gemm_fma_tiles(m->cfg.vocab);
#endif
  return gemm_tc_tiles(m->cfg.vocab);
}

Workspace carve_workspace(const specasr_model* m, int n_alloc, void* base) {
  const specasr_model_config& c = m->cfg;
  Workspace w;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    char* p = base ? (char*)base + off : nullptr;
    off += align_up(bytes, 256);
    return (void*)p;
  };
  const size_t wide = (size_t)(c.d_model > m->qkv_dim ? c.d_model : m->qkv_dim);
  w.ctl = (int32_t*)take(sizeof(int32_t) * kCtlWords);
  w.depth = (int32_t*)take(sizeof(int32_t) * n_alloc);
  w.pos = (int32_t*)take(sizeof(int32_t) * n_alloc);
  w.anc = (unsigned long long*)take(sizeof(unsigned long long) * 4 * n_alloc);
  w.X = (float*)take(sizeof(float) * n_alloc * c.d_model);
  w.H = (bf16*)take(sizeof(bf16) * 2 * n_alloc * c.d_model);
  w.P = (float*)take(sizeof(float) * kMaxSplitK * n_alloc * wide);
  w.fixP = (float*)take(m->cfg.gemm_path == 0 ? gemm_tc_fixup_bytes(m, n_alloc) : 256);
  w.fixFlag = (int32_t*)take(sizeof(int32_t) * (m->n_sm > 0 ? m->n_sm : 1));
  w.Q = (bf16*)take(sizeof(bf16) * 2 * n_alloc * m->q_dim);
  w.AO = (bf16*)take(sizeof(bf16) * 2 * n_alloc * m->q_dim);
  w.A = (bf16*)take(sizeof(bf16) * 2 * n_alloc * c.ffn);
  w.attO = (float*)take(sizeof(float) * kMaxAttnSplits * n_alloc * c.n_heads * c.head_dim);
  w.attML = (float2*)take(sizeof(float2) * kMaxAttnSplits * n_alloc * c.n_heads);
  w.amax = (unsigned long long*)take(sizeof(unsigned long long) * lm_tiles_of(m) * n_alloc);
  w.tmKV = (CUtensorMap*)take(sizeof(CUtensorMap) * 2);
  w.sec = (unsigned long long*)take(sizeof(unsigned long long) * lm_tiles_of(m) * n_alloc);
  w.lse = (float2*)take(sizeof(float2) * lm_tiles_of(m) * n_alloc);
  w.ssq = (float*)take(sizeof(float) * 2 * n_alloc);
  w.sync = (int32_t*)take(fused_stack_sync_bytes(m));
  w.bytes = off;
  return w;
}

// ------------------------------------------------------------------------------------------------
extern "C" void specasr_model_destroy(specasr_model* m);
static thread_local specasr_model* g_creating = nullptr;   // handle under construction, for the catch block below

static specasr_status model_create_impl(const specasr_model_config* cfg, const specasr_weight_ptrs* w,
                                        specasr_model** out) {
  if (!cfg || !w || !out) {
    set_error("specasr_model_create: null argument");
    return SPECASR_ERR_INVALID_ARG;
  }
  *out = nullptr;
  const specasr_model_config& c = *cfg;
  if (c.n_layers < 1 || c.d_model < 8 || c.n_heads < 1 || c.n_kv_heads < 1 || c.ffn < 8 || c.vocab < 1 ||
      c.max_positions < 1 || c.page_size < 1) {
    set_error("specasr_model_create: non-positive dimension");
    return SPECASR_ERR_INVALID_ARG;
  }
  if ((c.head_dim != 32 && c.head_dim != 64 && c.head_dim != 128) || c.n_heads % c.n_kv_heads != 0 ||
      c.d_model % 8 != 0 || c.ffn % 8 != 0 || c.page_size % 8 != 0 || (c.gemm_path != 0 && c.gemm_path != 1)) {
    set_error("specasr_model_create: unsupported shape (head_dim in {32,64,128}, d_model/ffn/page_size %% 8 == 0)");
    return SPECASR_ERR_UNSUPPORTED;
  }
#ifndef SPECASR_CROSSCHECK
  if (c.gemm_path != 0 || (c.head_dim != 64 && c.head_dim != 128) || c.page_size % 16 != 0 || c.page_size > 208 ||
      c.n_heads / c.n_kv_heads > 128) {
    set_error("specasr_model_create: this library has the tensor-core path only (gemm_path 0, head_dim 64 or 128, "
              "page_size a multiple of 16 up to 208, at most 128 query heads per KV head); other shapes exist in the "
              "cross-check build variant");
    return SPECASR_ERR_UNSUPPORTED;
  }
#endif
  if (!w->embed || !w->lm_head || !w->g_final || !w->wqkv || !w->wo || !w->wgu || !w->wd || !w->g_attn || !w->g_ffn) {
    set_error("specasr_model_create: null weight pointer");
    return SPECASR_ERR_INVALID_ARG;
  }
  specasr_model* m = new (std::nothrow) specasr_model();
  if (!m) {
    set_error("out of host memory");
    return SPECASR_ERR_INVALID_ARG;
  }
  g_creating = m;
  m->cfg = c;
  m->q_dim = c.n_heads * c.head_dim;
  m->kv_dim = c.n_kv_heads * c.head_dim;
  m->qkv_dim = m->q_dim + 2 * m->kv_dim;
  m->embed = (const bf16*)w->embed;
  m->lm_head = (const bf16*)w->lm_head;
  m->g_final = w->g_final;
  m->rope_table = nullptr;
  m->w_maps_dev = nullptr;
  m->gains_dev = nullptr;
  for (int l = 0; l < c.n_layers; ++l) {
    if (!w->wqkv[l] || !w->wo[l] || !w->wgu[l] || !w->wd[l] || !w->g_attn[l] || !w->g_ffn[l]) {
      delete m;
      set_error("specasr_model_create: null weight pointer in layer %d", l);
      return SPECASR_ERR_INVALID_ARG;
    }
    m->wqkv.push_back((const bf16*)w->wqkv[l]);
    m->wo.push_back((const bf16*)w->wo[l]);
    m->wgu.push_back((const bf16*)w->wgu[l]);
    m->wd.push_back((const bf16*)w->wd[l]);
    m->g_attn.push_back(w->g_attn[l]);
    m->g_ffn.push_back(w->g_ffn[l]);
  }
  cudaError_t e = cudaGetDevice(&m->device);
  cudaDeviceProp prop;
  if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, m->device);
  if (e != cudaSuccess) {
    delete m;
    set_error("no usable CUDA device: %s", cudaGetErrorString(e));
    return SPECASR_ERR_CUDA;
  }
  m->n_sm = prop.multiProcessorCount;
  if (c.gemm_path == 0 && prop.major != 10) {
    delete m;
    set_error("the tensor-core path needs an sm_100 device (found sm_%d%d)", prop.major, prop.minor);
    return SPECASR_ERR_UNSUPPORTED;
  }
  // rotary table in fp64 on the host: angle = pos * base^(-2k/dh)
  const int half = c.head_dim / 2;
  std::vector<float2> tab((size_t)c.max_positions * half);
  for (int k = 0; k < half; ++k) {
    const double theta = pow((double)c.rope_base, -2.0 * k / c.head_dim);
    for (int p = 0; p < c.max_positions; ++p) {
      const double ang = (double)p * theta;
      tab[(size_t)p * half + k] = make_float2((float)cos(ang), (float)sin(ang));
    }
  }
  e = cudaMalloc(&m->rope_table, tab.size() * sizeof(float2));
  if (e == cudaSuccess) e = cudaMemcpy(m->rope_table, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    if (m->rope_table) cudaFree(m->rope_table);
    delete m;
    set_error("rotary table upload failed: %s", cudaGetErrorString(e));
    return SPECASR_ERR_CUDA;
  }
  if (c.gemm_path == 0) {
    bool ok = true;
    m->tm_wqkv.resize(c.n_layers);
    m->tm_wo.resize(c.n_layers);
    m->tm_wgu.resize(c.n_layers);
    m->tm_wd.resize(c.n_layers);
    // tile-packed weights: a [M, K] matrix is a stack of 128 x 64 tiles, 128 bytes per row, one box per tile
    auto weight_map = [](CUtensorMap* map, const bf16* w, int K, uint64_t M) {
      const uint64_t rows = ((M + 127) / 128) * (uint64_t)packed_col_tiles(K) * 128;
      return make_tensor_map_2d(map, w, 64, rows, 64, 128);
    };
    for (int l = 0; l < c.n_layers && ok; ++l) {
      ok = ok && weight_map(&m->tm_wqkv[l], m->wqkv[l], c.d_model, m->qkv_dim);
      ok = ok && weight_map(&m->tm_wo[l], m->wo[l], m->q_dim, c.d_model);
      ok = ok && weight_map(&m->tm_wgu[l], m->wgu[l], c.d_model, 2 * (uint64_t)c.ffn);
      ok = ok && weight_map(&m->tm_wd[l], m->wd[l], c.ffn, c.d_model);
    }
    ok = ok && weight_map(&m->tm_lm, m->lm_head, c.d_model, c.vocab);
    if (!ok) {
      cudaFree(m->rope_table);
      delete m;
      return SPECASR_ERR_CUDA;   // message set by make_tensor_map_2d
    }
    // device copies of the weight descriptors and gain pointers, in the order the fused stack kernel walks them
    std::vector<CUtensorMap> maps;
    std::vector<const float*> gains;
    for (int l = 0; l < c.n_layers; ++l) {
      maps.push_back(m->tm_wqkv[l]);
      maps.push_back(m->tm_wo[l]);
      maps.push_back(m->tm_wgu[l]);
      maps.push_back(m->tm_wd[l]);
      gains.push_back(m->g_attn[l]);
      gains.push_back(m->g_ffn[l]);
    }
    maps.push_back(m->tm_lm);
    gains.push_back(m->g_final);
    e = cudaMalloc(&m->w_maps_dev, maps.size() * sizeof(CUtensorMap));
    if (e == cudaSuccess) e = cudaMalloc(&m->gains_dev, gains.size() * sizeof(const float*));
    if (e == cudaSuccess)
      e = cudaMemcpy(m->w_maps_dev, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
      e = cudaMemcpy(m->gains_dev, gains.data(), gains.size() * sizeof(const float*), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
      if (m->w_maps_dev) cudaFree(m->w_maps_dev);
      if (m->gains_dev) cudaFree(m->gains_dev);
      cudaFree(m->rope_table);
      delete m;
      set_error("descriptor upload failed: %s", cudaGetErrorString(e));
      return SPECASR_ERR_CUDA;
    }
  }
  *out = m;
  return SPECASR_OK;
}

// No C++ exception crosses the boundary: the handle's vectors can throw std::bad_alloc.
extern "C" specasr_status specasr_model_create(const specasr_model_config* cfg, const specasr_weight_ptrs* w,
                                               specasr_model** out) {
  g_creating = nullptr;
  try {
    const specasr_status st = model_create_impl(cfg, w, out);
    g_creating = nullptr;
    return st;
  } catch (...) {
    if (out) *out = nullptr;
    if (g_creating) specasr_model_destroy(g_creating);
    g_creating = nullptr;
    set_error("specasr_model_create: out of host memory");
    return SPECASR_ERR_INVALID_ARG;
  }
}

extern "C" void specasr_model_destroy(specasr_model* m) {
  if (!m) return;
  if (m->rope_table) cudaFree(m->rope_table);
  if (m->w_maps_dev) cudaFree(m->w_maps_dev);
  if (m->gains_dev) cudaFree(m->gains_dev);
  delete m;
}

extern "C" size_t specasr_workspace_bytes(const specasr_model* m, int32_t max_nodes) {
  if (!m || max_nodes < 1 || max_nodes > SPECASR_MAX_NODES) return 0;
  return carve_workspace(m, pad_tokens(max_nodes), nullptr).bytes;
}

extern "C" size_t specasr_kv_pool_bytes(const specasr_model* m, int32_t n_pages) {
  if (!m || n_pages < 1) return 0;
  const specasr_model_config& c = m->cfg;
  return (size_t)c.n_layers * n_pages * c.n_kv_heads * 2 * c.page_size * c.head_dim * sizeof(bf16);
}

extern "C" specasr_status specasr_kv_create(const specasr_model* m, void* k_pool, void* v_pool, int32_t n_pages,
                                            const int32_t* page_table, int32_t max_pages, void* workspace,
                                            int32_t max_nodes, specasr_kv** out) {
  if (!m || !k_pool || !v_pool || !page_table || !workspace || !out) {
    set_error("specasr_kv_create: null argument");
    return SPECASR_ERR_INVALID_ARG;
  }
  *out = nullptr;
  if (n_pages < 1 || max_pages < 1 || max_nodes < 1 || max_nodes > SPECASR_MAX_NODES) {
    set_error("specasr_kv_create: n_pages, max_pages >= 1 and 1 <= max_nodes <= %d required", SPECASR_MAX_NODES);
    return SPECASR_ERR_INVALID_ARG;
  }
  if (((uintptr_t)workspace & 255) || ((uintptr_t)k_pool & 15) || ((uintptr_t)v_pool & 15)) {
    set_error("specasr_kv_create: workspace must be 256-byte aligned, pools 16-byte aligned");
    return SPECASR_ERR_INVALID_ARG;
  }
  specasr_kv* kv = new (std::nothrow) specasr_kv();
  if (!kv) {
    set_error("out of host memory");
    return SPECASR_ERR_INVALID_ARG;
  }
  kv->m = m;
  kv->k_pool = (bf16*)k_pool;
  kv->v_pool = (bf16*)v_pool;
  kv->n_pages = n_pages;
  kv->page_table = page_table;
  kv->max_pages = max_pages;
  kv->max_nodes = max_nodes;
  kv->n_alloc = pad_tokens(max_nodes);
  kv->ws = carve_workspace(m, kv->n_alloc, workspace);
  kv->pending_n = 0;
  kv->len_host = 0;
  kv->len_exact = true;
  kv->len_upper = 0;
  kv->pinned = nullptr;
  kv->len_event_pending = false;
  kv->launches = 0;
  kv->gemm_epoch = 0;
  kv->prof_on = false;
  kv->prof_used = 0;
  kv->attn_tc = false;
  kv->trace.buf = nullptr;
  kv->trace.cap = 0;
  cudaError_t e = cudaHostAlloc(&kv->pinned, 4 * sizeof(int32_t), cudaHostAllocDefault);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&kv->len_event, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaMemset(kv->ws.ctl, 0, sizeof(int32_t) * kCtlWords);
  if (e == cudaSuccess) e = cudaMemset(kv->ws.fixFlag, 0, sizeof(int32_t) * m->n_sm);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    if (kv->pinned) cudaFreeHost(kv->pinned);
    delete kv;
    set_error("specasr_kv_create: %s", cudaGetErrorString(e));
    return SPECASR_ERR_CUDA;
  }
  if (m->cfg.gemm_path == 0) {
    const specasr_model_config& c = m->cfg;
    bool ok = true;
    for (int i = 0, b = 16; i < 5 && b <= kv->n_alloc && ok; ++i, b <<= 1) {
      ok = make_act_map(&kv->tm_H[i], kv->ws.H, c.d_model, kv->n_alloc, b) &&
           make_act_map(&kv->tm_AO[i], kv->ws.AO, m->q_dim, kv->n_alloc, b) &&
           make_act_map(&kv->tm_A[i], kv->ws.A, c.ffn, kv->n_alloc, b);
    }
    kv->attn_tc = ok && attention_tc_supported(m);
    if (kv->attn_tc) ok = attention_tc_make_maps(kv);
    if (!ok) {
      cudaFreeHost(kv->pinned);
      cudaEventDestroy(kv->len_event);
      delete kv;
      return SPECASR_ERR_CUDA;
    }
  }
  *out = kv;
  return SPECASR_OK;
}

extern "C" void specasr_kv_destroy(specasr_kv* kv) {
  if (!kv) return;
  if (kv->len_event_pending) cudaEventSynchronize(kv->len_event);
  for (cudaEvent_t e : kv->prof_events) cudaEventDestroy(e);
  cudaEventDestroy(kv->len_event);
  if (kv->pinned) cudaFreeHost(kv->pinned);
  delete kv;
}

extern "C" int64_t specasr_launch_count(const specasr_kv* kv) { return kv ? kv->launches : 0; }

extern "C" specasr_status specasr_trace_set(specasr_kv* kv, void* buffer, int64_t capacity_records) {
  if (!kv || capacity_records < 0 || (buffer && ((uintptr_t)buffer & 7))) {
    set_error("specasr_trace_set: null handle, negative capacity or misaligned buffer");
    return SPECASR_ERR_INVALID_ARG;
  }
#ifndef SPECASR_TRACE
  if (buffer) {
    set_error("specasr_trace_set: this library was built without -DSPECASR_TRACE (use libspecasr_trace.so)");
    return SPECASR_ERR_UNSUPPORTED;
  }
#endif
  kv->trace.buf = (unsigned long long*)buffer;
  kv->trace.cap = buffer ? (unsigned long long)capacity_records : 0ull;
  return SPECASR_OK;
}

extern "C" specasr_status specasr_profile_enable(specasr_kv* kv, int32_t enable) {
  if (!kv) {
    set_error("specasr_profile_enable: null handle");
    return SPECASR_ERR_INVALID_ARG;
  }
  kv->prof_on = enable != 0;
  kv->prof_used = 0;
  return SPECASR_OK;
}

extern "C" specasr_status specasr_profile_read(specasr_kv* kv, double* out_ms, int64_t* out_launches, void* stream) {
  if (!kv || !out_ms || !out_launches) {
    set_error("specasr_profile_read: null argument");
    return SPECASR_ERR_INVALID_ARG;
  }
  CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
  for (int k = 0; k < SPECASR_KIND_COUNT; ++k) {
    out_ms[k] = 0.0;
    out_launches[k] = 0;
  }
  for (size_t i = 0; i < kv->prof_used; ++i) {
    float ms = 0.f;
    CUDA_TRY(cudaEventElapsedTime(&ms, kv->prof_events[2 * i], kv->prof_events[2 * i + 1]));
    out_ms[kv->prof_kinds[i]] += ms;
    out_launches[kv->prof_kinds[i]] += 1;
  }
  kv->prof_used = 0;
  return SPECASR_OK;
}

// The host learns the committed length lazily: a commit enqueues a copy of the device length word
// into pinned memory followed by an event.
static void refresh_len(specasr_kv* kv, bool wait) {
  if (!kv->len_event_pending) return;
  cudaError_t q = wait ? cudaEventSynchronize(kv->len_event) : cudaEventQuery(kv->len_event);
  if (q == cudaSuccess) {
    kv->len_host = kv->pinned[0];
    kv->len_upper = kv->len_host;
    kv->len_exact = true;
    kv->len_event_pending = false;
  } else if (q != cudaErrorNotReady) {
    cudaGetLastError();
  }
}

extern "C" specasr_status specasr_kv_length(specasr_kv* kv, int32_t* out_len, void* stream) {
  (void)stream;
  if (!kv || !out_len) {
    set_error("specasr_kv_length: null argument");
    return SPECASR_ERR_INVALID_ARG;
  }
  refresh_len(kv, true);
  *out_len = kv->len_host;
  return SPECASR_OK;
}

extern "C" specasr_status specasr_kv_truncate(specasr_kv* kv, int32_t len, void* stream) {
  if (!kv) {
    set_error("specasr_kv_truncate: null handle");
    return SPECASR_ERR_INVALID_ARG;
  }
  refresh_len(kv, true);
  if (len < 0 || len > kv->len_host) {
    set_error("specasr_kv_truncate: len %d outside [0, %d]", len, kv->len_host);
    return SPECASR_ERR_INVALID_ARG;
  }
  launch_set_len(kv, len, (cudaStream_t)stream);
  kv->len_host = kv->len_upper = len;
  kv->pending_n = 0;
  CUDA_TRY(cudaGetLastError());
  return SPECASR_OK;
}

extern "C" specasr_status specasr_poll_status(specasr_kv* kv, int32_t* out_device_status, void* stream) {
  if (!kv || !out_device_status) {
    set_error("specasr_poll_status: null argument");
    return SPECASR_ERR_INVALID_ARG;
  }
  cudaStream_t s = (cudaStream_t)stream;
  CUDA_TRY(cudaMemcpyAsync(kv->pinned + 2, kv->ws.ctl + CTL_STATUS, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaStreamSynchronize(s));
  *out_device_status = kv->pinned[2];
  return SPECASR_OK;
}

// ------------------------------------------------------------------------------------------------
static void run_gemm(specasr_kv* kv, GemmArgs& a, int kind, cudaStream_t s) {
#ifdef SPECASR_CROSSCHECK
  if (kv->m->cfg.gemm_path == 1) {
    a.splits = 1;
    launch_gemm_fma(kv, a, kind, s);
    return;
  }
#endif
  a.splits = gemm_tc_pick_splits(kv->m, a.M, a.K, a.n_pad);
  launch_gemm_tc(kv, a, kind, s);
}

// Key blocks of the attention over `n` nodes of one utterance; `sm_budget` is the number of SMs the launch
// should fill (all of them for a plain call, a share of them when several utterances launch back to back).
static int attention_splits(const specasr_kv* kv, int n, int len_upper, int sm_budget, bool* use_tc, int* chunk) {
  const specasr_model_config& c = kv->m->cfg;
  *use_tc = false;
  *chunk = 0;
  if (kv->attn_tc) {
    int s = 0;
    if (attention_tc_plan(kv->m, n, len_upper + n, sm_budget, kMaxAttnSplits, &s, chunk)) {
      *use_tc = true;
      return s;
    }
  }
  const int group = c.n_heads / c.n_kv_heads;
  const int row_tiles = (n * group + 63) / 64;
  const int ctas = c.n_kv_heads * row_tiles;
  int splits = (sm_budget + ctas - 1) / ctas;
  const int by_len = (len_upper + n + 63) / 64;
  if (splits > by_len) splits = by_len;
  if (splits > kMaxAttnSplits) splits = kMaxAttnSplits;
  if (splits < 1) splits = 1;
  return splits;
}

// Table entry of one utterance (everything but the attention plan).
static SegDev seg_entry(const specasr_kv* u, int row0, int n) {
  SegDev d;
  memset(&d, 0, sizeof(d));
  d.ctl = u->ws.ctl;
  d.page_table = u->page_table;
  d.k_pool = u->k_pool;
  d.v_pool = u->v_pool;
  d.tmK = u->attn_tc ? u->ws.tmKV : nullptr;
  d.tmV = u->attn_tc ? u->ws.tmKV + 1 : nullptr;
  d.n_pages = u->n_pages;
  d.row0 = row0;
  d.n = n;
  int cap = u->max_pages * u->m->cfg.page_size;
  if (u->m->cfg.max_positions < cap) cap = u->m->cfg.max_positions;
  d.capacity = cap;
  return d;
}

// The layer stack over the rows of the utterances in `tab`, laid out back to back in the workspace of `wk`
// (n_total rows, layer-0 inputs already in ws.X).  Norms, projections and the attention merge look at the
// control block `ctl_shared`; the rotary/append and attention kernels look up each row's utterance in the table
// and work against its cache and control block.  With want_head the final norm, the vocabulary projection
// and its fused per-tile argmax run as well.
static void run_stack(specasr_model* m, specasr_kv* wk, const SegTable& tab, int n_total, int n_max, bool att_tc,
                      const int32_t* ctl_shared, bool want_head, float* out_logits, bool want_top2, cudaStream_t s) {
  const specasr_model_config& c = m->cfg;
  const int n = n_total;
  if (fused_stack_supported(wk, n_total, att_tc, tab.splits)) {
    launch_fused_stack(m, wk, tab, n_total, n_max, ctl_shared, want_head, out_logits, want_top2, s);
    return;
  }
  const int n_pad = pad_tokens(n);
  const bool tc = c.gemm_path == 0;
  int pending = 0;               // partial planes of the last down projection still to be added to X
  GemmArgs a;
  memset(&a, 0, sizeof(a));
  a.n = n;
  a.n_pad = n_pad;
  a.n_alloc = wk->n_alloc;
  a.ctl = ctl_shared;
  a.P = wk->ws.P;
  for (int l = 0; l < c.n_layers; ++l) {
    launch_rmsnorm_split(wk, ctl_shared, m->g_attn[l], n, n_pad, pending, s);
    a.W = m->wqkv[l]; a.tmW = tc ? &m->tm_wqkv[l] : nullptr; a.tmAct = wk->tm_H; a.act = wk->ws.H;
    a.M = m->qkv_dim; a.K = c.d_model; a.epilogue = EPI_PARTIAL;
    run_gemm(wk, a, SPECASR_KIND_GEMM_QKV, s);
    launch_rope_append(wk, tab, n, l, a.splits, s);
#ifdef SPECASR_CROSSCHECK
    if (!att_tc) launch_tree_attention(wk, l, n, tab.splits, s);      // plain kernel, single utterance only
    else
#endif
      launch_tree_attention_tc(wk, tab, n_max, l, s);
    launch_attn_merge(wk, ctl_shared, n, n_pad, tab.splits, s);
    a.W = m->wo[l]; a.tmW = tc ? &m->tm_wo[l] : nullptr; a.tmAct = wk->tm_AO; a.act = wk->ws.AO;
    a.M = c.d_model; a.K = m->q_dim; a.epilogue = EPI_PARTIAL;
    run_gemm(wk, a, SPECASR_KIND_GEMM_O, s);
    launch_rmsnorm_split(wk, ctl_shared, m->g_ffn[l], n, n_pad, a.splits, s);
    a.W = m->wgu[l]; a.tmW = tc ? &m->tm_wgu[l] : nullptr; a.tmAct = wk->tm_H; a.act = wk->ws.H;
    a.M = 2 * c.ffn; a.K = c.d_model; a.epilogue = EPI_SWIGLU; a.A = wk->ws.A;
    run_gemm(wk, a, SPECASR_KIND_GEMM_GU, s);
    a.W = m->wd[l]; a.tmW = tc ? &m->tm_wd[l] : nullptr; a.tmAct = wk->tm_A; a.act = wk->ws.A;
    a.M = c.d_model; a.K = c.ffn; a.epilogue = EPI_PARTIAL;
    run_gemm(wk, a, SPECASR_KIND_GEMM_DOWN, s);
    pending = a.splits;
  }
  if (!want_head) return;   // context fill: K/V of every layer are written, the last FFN output is not needed
  launch_rmsnorm_split(wk, ctl_shared, m->g_final, n, n_pad, pending, s);
  a.W = m->lm_head; a.tmW = tc ? &m->tm_lm : nullptr; a.tmAct = wk->tm_H; a.act = wk->ws.H;
  a.M = c.vocab; a.K = c.d_model; a.epilogue = EPI_ARGMAX; a.amax = wk->ws.amax; a.logits = out_logits;
  run_gemm(wk, a, SPECASR_KIND_GEMM_LM, s);
}

// The table of a plain call: one utterance at row 0 of its own workspace, attention planned for the whole GPU.
static SegTable single_table(specasr_kv* kv, int n, bool* att_tc) {
  SegTable t;
  memset(&t, 0, sizeof(t));
  t.count = 1;
  t.seg[0] = seg_entry(kv, 0, n);
  t.splits = attention_splits(kv, n, kv->len_upper, kv->m->n_sm, att_tc, &t.seg[0].chunk);
  return t;
}

static specasr_status prefill_common(specasr_model* m, specasr_kv* kv, const float* embeds, const int32_t* tokens,
                                     int n, cudaStream_t s, const char* who) {
  if (!m || !kv || (!embeds && !tokens)) {
    set_error("%s: null argument", who);
    return SPECASR_ERR_INVALID_ARG;
  }
  if (kv->m != m) {
    set_error("%s: KV handle belongs to another model", who);
    return SPECASR_ERR_INVALID_ARG;
  }
  if (n < 1) {
    set_error("%s: n must be >= 1", who);
    return SPECASR_ERR_INVALID_ARG;
  }
  refresh_len(kv, true);
  int cap = kv->max_pages * m->cfg.page_size;
  if (m->cfg.max_positions < cap) cap = m->cfg.max_positions;
  if (kv->len_host + n > cap) {
    set_error("%s: %d + %d positions exceed the capacity of %d", who, kv->len_host, n, cap);
    return SPECASR_ERR_KV_CAPACITY;
  }
  kv->pending_n = 0;
  for (int done = 0; done < n;) {
    const int chunk = n - done < kv->max_nodes ? n - done : kv->max_nodes;
    bool att_tc = false;
    const SegTable tab = single_table(kv, chunk, &att_tc);
#ifndef SPECASR_CROSSCHECK
    if (!att_tc) {
      set_error("%s: a cache of %d positions needs more key blocks than the workspace holds", who, kv->len_upper + chunk);
      return SPECASR_ERR_UNSUPPORTED;
    }
#endif
    launch_chain_prep(kv, chunk, done == 0, s);
    if (embeds) launch_copy_embeds(kv, embeds + (size_t)done * m->cfg.d_model, chunk, s);
    else launch_embed_tokens(kv, tab, chunk, tokens + done, s);
    run_stack(m, kv, tab, chunk, chunk, att_tc, kv->ws.ctl, false, nullptr, false, s);
    launch_advance_len(kv, chunk, s);
    kv->len_host += chunk;
    kv->len_upper = kv->len_host;
    done += chunk;
  }
  // The device may have refused a chunk (a token id outside the vocabulary): the host learns the length the same
  // lazy way as after a commit, so that specasr_kv_length reports what the device holds.
  CUDA_TRY(cudaMemcpyAsync(kv->pinned, kv->ws.ctl + CTL_LEN, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaEventRecord(kv->len_event, s));
  kv->len_event_pending = true;           // len_host stays the optimistic value (an upper bound) until the copy lands
  CUDA_TRY(cudaGetLastError());
  return SPECASR_OK;
}

extern "C" specasr_status specasr_prefill_embeds(specasr_model* m, specasr_kv* kv, const float* embeds, int32_t n,
                                                 void* stream) {
  return prefill_common(m, kv, embeds, nullptr, n, (cudaStream_t)stream, "specasr_prefill_embeds");
}

extern "C" specasr_status specasr_prefill_tokens(specasr_model* m, specasr_kv* kv, const int32_t* tokens, int32_t n,
                                                 void* stream) {
  return prefill_common(m, kv, nullptr, tokens, n, (cudaStream_t)stream, "specasr_prefill_tokens");
}

static specasr_status verify_tree_impl(specasr_model* m, specasr_kv* kv, const int32_t* tokens,
                                       const int32_t* parent_idx, int32_t n_nodes, int32_t* out_argmax,
                                       int32_t* out_accept_len, int32_t* out_path, float* out_logits,
                                       int32_t* out_bonus, int32_t* out_top2_ids, float* out_top2_probs, void* stream) {
  if (!m || !kv || !tokens || !parent_idx || !out_argmax || !out_accept_len || !out_path) {
    set_error("specasr_verify_tree: null argument");
    return SPECASR_ERR_INVALID_ARG;
  }
  if (kv->m != m) {
    set_error("specasr_verify_tree: KV handle belongs to another model");
    return SPECASR_ERR_INVALID_ARG;
  }
  if (n_nodes < 1 || n_nodes > kv->max_nodes) {
    set_error("specasr_verify_tree: n_nodes = %d outside [1, %d]", n_nodes, kv->max_nodes);
    return SPECASR_ERR_INVALID_ARG;
  }
  refresh_len(kv, false);
  int cap = kv->max_pages * m->cfg.page_size;
  if (m->cfg.max_positions < cap) cap = m->cfg.max_positions;
  if (kv->len_exact && kv->len_host + n_nodes > cap) {
    set_error("specasr_verify_tree: %d committed + %d tree slots exceed the capacity of %d", kv->len_host, n_nodes, cap);
    return SPECASR_ERR_KV_CAPACITY;
  }
  cudaStream_t s = (cudaStream_t)stream;
  bool att_tc = false;
  const SegTable tab = single_table(kv, n_nodes, &att_tc);
#ifndef SPECASR_CROSSCHECK
  if (!att_tc) {
    set_error("specasr_verify_tree: a cache of %d positions needs more key blocks than the workspace holds",
              kv->len_upper + n_nodes);
    return SPECASR_ERR_UNSUPPORTED;
  }
#endif
  const bool want_top2 = out_top2_ids != nullptr;
  if (want_top2 && !fused_stack_supported(kv, n_nodes, att_tc, tab.splits)) {
    set_error("specasr_verify_tree_top2: the top-2 epilogue needs the fused layer stack (tensor-core attention, at most "
              "64 nodes)");
    return SPECASR_ERR_UNSUPPORTED;
  }
  launch_tree_prep(kv, tab, tokens, parent_idx, s);
  launch_embed_tokens(kv, tab, n_nodes, tokens, s);
  run_stack(m, kv, tab, n_nodes, n_nodes, att_tc, kv->ws.ctl, true, out_logits, want_top2, s);
  launch_accept(kv, tab, nullptr, tokens, parent_idx, lm_tiles_of(m), out_argmax, out_accept_len, out_path, out_bonus, s);
  if (want_top2) launch_top2_from_tiles(kv, tab, nullptr, n_nodes, lm_tiles_of(m), out_top2_ids, out_top2_probs, s);
  kv->pending_n = n_nodes;
  CUDA_TRY(cudaGetLastError());
  return SPECASR_OK;
}

extern "C" specasr_status specasr_verify_tree_ex(specasr_model* m, specasr_kv* kv, const int32_t* tokens,
                                                 const int32_t* parent_idx, int32_t n_nodes, int32_t* out_argmax,
                                                 int32_t* out_accept_len, int32_t* out_path, float* out_logits,
                                                 int32_t* out_bonus, void* stream) {
  return verify_tree_impl(m, kv, tokens, parent_idx, n_nodes, out_argmax, out_accept_len, out_path, out_logits,
                          out_bonus, nullptr, nullptr, stream);
}

extern "C" specasr_status specasr_verify_tree_top2(specasr_model* m, specasr_kv* kv, const int32_t* tokens,
                                                   const int32_t* parent_idx, int32_t n_nodes, int32_t* out_argmax,
                                                   int32_t* out_accept_len, int32_t* out_path, int32_t* out_bonus,
                                                   int32_t* out_top2_ids, float* out_top2_probs, void* stream) {
  if (!out_top2_ids || !out_top2_probs) {
    set_error("specasr_verify_tree_top2: null output");
    return SPECASR_ERR_INVALID_ARG;
  }
  return verify_tree_impl(m, kv, tokens, parent_idx, n_nodes, out_argmax, out_accept_len, out_path, nullptr, out_bonus,
                          out_top2_ids, out_top2_probs, stream);
}

extern "C" specasr_status specasr_verify_tree(specasr_model* m, specasr_kv* kv, const int32_t* tokens,
                                              const int32_t* parent_idx, int32_t n_nodes, int32_t* out_argmax,
                                              int32_t* out_accept_len, int32_t* out_path, void* stream) {
  return specasr_verify_tree_ex(m, kv, tokens, parent_idx, n_nodes, out_argmax, out_accept_len, out_path, nullptr,
                                nullptr, stream);
}

// Several utterances in one pass over the weights: the verification of Section II-B applied to each utterance,
// with the norms and projections run once over all rows.
static specasr_status verify_batch_impl(specasr_model* m, int32_t batch, specasr_kv* const* kv,
                                        const int32_t* tokens, const int32_t* parent_idx,
                                        const int32_t* node_offsets, int32_t* out_argmax,
                                        int32_t* out_accept_len, int32_t* out_path, float* out_logits,
                                        int32_t* out_bonus, int32_t* out_top2_ids, float* out_top2_probs, void* stream) {
  const char* who = "specasr_verify_tree_batch";
  if (!m || !kv || !tokens || !parent_idx || !node_offsets || !out_argmax || !out_accept_len || !out_path) {
    set_error("%s: null argument", who);
    return SPECASR_ERR_INVALID_ARG;
  }
  if (batch < 1 || batch > SPECASR_MAX_BATCH) {
    set_error("%s: batch = %d outside [1, %d]", who, batch, SPECASR_MAX_BATCH);
    return SPECASR_ERR_INVALID_ARG;
  }
  if (node_offsets[0] != 0) {
    set_error("%s: node_offsets[0] must be 0", who);
    return SPECASR_ERR_INVALID_ARG;
  }
  for (int b = 0; b < batch; ++b) {
    if (!kv[b] || kv[b]->m != m) {
      set_error("%s: handle %d is null or belongs to another model", who, b);
      return SPECASR_ERR_INVALID_ARG;
    }
    for (int j = 0; j < b; ++j)
      if (kv[j] == kv[b]) {
        set_error("%s: handle %d appears twice", who, b);
        return SPECASR_ERR_INVALID_ARG;
      }
    if (node_offsets[b + 1] <= node_offsets[b]) {
      set_error("%s: utterance %d has no nodes (node_offsets must increase)", who, b);
      return SPECASR_ERR_INVALID_ARG;
    }
  }
  specasr_kv* wk = kv[0];
  const int total = node_offsets[batch];
  if (total > wk->max_nodes) {
    set_error("%s: %d nodes in all exceed the %d rows of the first handle's workspace", who, total, wk->max_nodes);
    return SPECASR_ERR_INVALID_ARG;
  }
  SegTable tab;
  memset(&tab, 0, sizeof(tab));
  tab.count = batch;
  tab.splits = 1;
  int budget = m->n_sm / batch;
  if (budget < 1) budget = 1;
  int n_max = 1;
  for (int b = 0; b < batch; ++b) {
    specasr_kv* u = kv[b];
    const int n_b = node_offsets[b + 1] - node_offsets[b];
    if (!u->attn_tc) {
      set_error("%s: needs the tensor-core attention path (head_dim 64 or 128, page_size %% 16 == 0)", who);
      return SPECASR_ERR_UNSUPPORTED;
    }
    refresh_len(u, false);
    tab.seg[b] = seg_entry(u, node_offsets[b], n_b);
    if (u->len_exact && u->len_host + n_b > tab.seg[b].capacity) {
      set_error("%s: utterance %d: %d committed + %d tree slots exceed the capacity of %d", who, b, u->len_host, n_b,
                tab.seg[b].capacity);
      return SPECASR_ERR_KV_CAPACITY;
    }
    bool use_tc = false;
    const int sp = attention_splits(u, n_b, u->len_upper, budget, &use_tc, &tab.seg[b].chunk);
    if (!use_tc) {
      set_error("%s: utterance %d: cache of up to %d positions needs more key blocks than the workspace holds", who, b,
                u->len_upper + n_b);
      return SPECASR_ERR_UNSUPPORTED;
    }
    if (sp > tab.splits) tab.splits = sp;
    if (n_b > n_max) n_max = n_b;
  }
  cudaStream_t s = (cudaStream_t)stream;
  int32_t* ctl_shared = wk->ws.ctl + kCtlBatch;
  CUDA_TRY(cudaMemsetAsync(ctl_shared, 0, sizeof(int32_t) * 4, s));
  const bool want_top2 = out_top2_ids != nullptr;
  if (want_top2 && !fused_stack_supported(wk, total, true, tab.splits)) {
    set_error("%s: the top-2 epilogue needs the fused layer stack (at most 64 nodes in all)", who);
    return SPECASR_ERR_UNSUPPORTED;
  }
  launch_tree_prep(wk, tab, tokens, parent_idx, s);
  launch_embed_tokens(wk, tab, total, tokens, s);
  run_stack(m, wk, tab, total, n_max, true, ctl_shared, true, out_logits, want_top2, s);
  launch_accept(wk, tab, ctl_shared, tokens, parent_idx, lm_tiles_of(m), out_argmax, out_accept_len, out_path, out_bonus,
                s);
  if (want_top2) launch_top2_from_tiles(wk, tab, ctl_shared, total, lm_tiles_of(m), out_top2_ids, out_top2_probs, s);
  for (int b = 0; b < batch; ++b) kv[b]->pending_n = tab.seg[b].n;
  CUDA_TRY(cudaGetLastError());
  return SPECASR_OK;
}

extern "C" specasr_status specasr_verify_tree_batch(specasr_model* m, int32_t batch, specasr_kv* const* kv,
                                                    const int32_t* tokens, const int32_t* parent_idx,
                                                    const int32_t* node_offsets, int32_t* out_argmax,
                                                    int32_t* out_accept_len, int32_t* out_path, float* out_logits,
                                                    int32_t* out_bonus, void* stream) {
  return verify_batch_impl(m, batch, kv, tokens, parent_idx, node_offsets, out_argmax, out_accept_len, out_path,
                           out_logits, out_bonus, nullptr, nullptr, stream);
}

extern "C" specasr_status specasr_verify_tree_batch_top2(specasr_model* m, int32_t batch, specasr_kv* const* kv,
                                                         const int32_t* tokens, const int32_t* parent_idx,
                                                         const int32_t* node_offsets, int32_t* out_argmax,
                                                         int32_t* out_accept_len, int32_t* out_path, int32_t* out_bonus,
                                                         int32_t* out_top2_ids, float* out_top2_probs, void* stream) {
  if (!out_top2_ids || !out_top2_probs) {
    set_error("specasr_verify_tree_batch_top2: null output");
    return SPECASR_ERR_INVALID_ARG;
  }
  return verify_batch_impl(m, batch, kv, tokens, parent_idx, node_offsets, out_argmax, out_accept_len, out_path, nullptr,
                           out_bonus, out_top2_ids, out_top2_probs, stream);
}

extern "C" specasr_status specasr_commit_kv(specasr_model* m, specasr_kv* kv, const int32_t* path,
                                            const int32_t* accept_len, void* stream) {
  if (!m || !kv || !path || !accept_len) {
    set_error("specasr_commit_kv: null argument");
    return SPECASR_ERR_INVALID_ARG;
  }
  if (kv->m != m) {
    set_error("specasr_commit_kv: KV handle belongs to another model");
    return SPECASR_ERR_INVALID_ARG;
  }
  if (kv->pending_n == 0) {
    set_error("specasr_commit_kv: no verify is pending on this handle");
    return SPECASR_ERR_STATE;
  }
  cudaStream_t s = (cudaStream_t)stream;
  refresh_len(kv, false);
  launch_commit(kv, path, accept_len, s);
  CUDA_TRY(cudaMemcpyAsync(kv->pinned, kv->ws.ctl + CTL_LEN, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaEventRecord(kv->len_event, s));
  kv->len_event_pending = true;
  kv->len_exact = false;
  kv->len_upper += kv->pending_n;
  kv->pending_n = 0;
  CUDA_TRY(cudaGetLastError());
  return SPECASR_OK;
}
