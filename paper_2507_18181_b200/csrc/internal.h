// Internal declarations of the tree-verification library (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <vector>

#include "specasr.h"

typedef __nv_bfloat16 bf16;

constexpr int kMaxSplitK = 12;     // partial planes of the linear projections
constexpr int kMaxAttnSplits = 40; // KV splits of the attention kernels
constexpr int kCtlWords = 64;      // int32 control block at the start of the workspace

// control block word indices
enum { CTL_LEN = 0, CTL_STATUS = 1, CTL_N = 2 };
// A second control block (same word layout) at this offset serves the kernels that a batched call runs once
// over all utterances: its status word only ever records a bounded wait that ran out.
constexpr int kCtlBatch = 16;

// Optional device-side trace (specasr_trace_set): every thread block of the traced kernels appends one record
// {kind, start, end, time its wait for the previous kernel ended} of %globaltimer nanoseconds.  Event pairs around
// a launch switch the overlap of consecutive kernels off; these stamps do not.
struct TraceBuf {
  unsigned long long* buf;  // [0] = records written so far, [1] unused, records of 4 words from [2]; null = off
  unsigned long long cap;   // records the buffer holds
};

// The trace exists only in the library variant built with -DSPECASR_TRACE; in the product build these expand to
// nothing, so that kernel signatures, parameter structs and register allocation are exactly those without it.
#ifdef SPECASR_TRACE
#define SPECASR_TRACE_PARAM , TraceBuf tr
#define SPECASR_TRACE_ARG(kv) , (kv)->trace
#define SPECASR_TRACE_SCOPE(tr, kind) TraceScope trace_(tr, kind)
#define SPECASR_TRACE_MARK() trace_.mark()
#else
#define SPECASR_TRACE_PARAM
#define SPECASR_TRACE_ARG(kv)
#define SPECASR_TRACE_SCOPE(tr, kind)
#define SPECASR_TRACE_MARK()
#endif

struct specasr_model {
  specasr_model_config cfg;
  int device;
  int qkv_dim;              // (Hq + 2 Hkv) * dh
  int q_dim;                // Hq * dh
  int kv_dim;               // Hkv * dh
  const bf16* embed;
  const bf16* lm_head;
  const float* g_final;
  std::vector<const bf16*> wqkv, wo, wgu, wd;
  std::vector<const float*> g_attn, g_ffn;
  float2* rope_table;       // [max_positions][dh/2] (cos, sin), built in fp64 on the host
  std::vector<CUtensorMap> tm_wqkv, tm_wo, tm_wgu, tm_wd;
  CUtensorMap tm_lm;
  CUtensorMap* w_maps_dev;  // device copy for the fused layer-stack kernel: [4 * layers + 1] QKV, O, gate/up, down, ..., vocabulary
  const float** gains_dev;  // device array [2 * layers + 1]: attention / FFN norm gains per layer, then the final norm
  int n_sm;
};

struct Workspace {
  int32_t* ctl;             // [kCtlWords]
  int32_t* depth;           // [n_alloc]
  int32_t* pos;             // [n_alloc]
  unsigned long long* anc;  // [n_alloc][4] ancestor-or-self bitmask over node indices
  float* X;                 // [n_alloc][d] residual stream
  bf16* H;                  // [2][n_alloc][d]      normed activations, hi / lo planes
  float* P;                 // [kMaxSplitK][n_alloc][max(d, qkv_dim)] partial sums of the linear projections
  float* fixP;              // [n_sm][n_alloc][128] partial tiles of the persistent tensor-core projections
  int32_t* fixFlag;         // [n_sm] launch number of the partial tile each CTA published last
  bf16* Q;                  // [2][n_alloc][q_dim]  rotated queries, hi / lo planes
  bf16* AO;                 // [2][n_alloc][q_dim]  attention output, hi / lo planes
  bf16* A;                  // [2][n_alloc][ffn]    SwiGLU output, hi / lo planes
  float* attO;              // [kMaxAttnSplits][n_alloc * Hq][dh] unnormalised partial outputs
  float2* attML;            // [kMaxAttnSplits][n_alloc * Hq]     (running max in log2 units, sum)
  unsigned long long* amax; // [lm_tiles][n_alloc] packed (ordered logit, ~token id) per vocab tile
  CUtensorMap* tmKV;        // [2] device copies of the K and V pool descriptors (tensor-core attention)
  unsigned long long* sec;  // [lm_tiles][n_alloc] second-best packed key per vocabulary tile (fused stack, on request)
  float2* lse;              // [lm_tiles][n_alloc] (max, sum of exp) per vocabulary tile (fused stack, on request)
  float* ssq;               // [2][n_alloc] sums of squares of the two halves of every residual row (fused stack)
  int32_t* sync;            // arrival counters of the fused stack kernel, one per step of the call
  size_t bytes;
};

struct specasr_kv {
  const specasr_model* m;
  bf16* k_pool;
  bf16* v_pool;
  int n_pages;
  const int32_t* page_table;
  int max_pages;
  int max_nodes;
  int n_alloc;              // max_nodes rounded up to 16
  Workspace ws;
  // host-side state
  int pending_n;            // nodes of the verify awaiting a commit, 0 = none
  int len_host;             // last length the host knows exactly
  bool len_exact;           // false while a commit's length has not been read back
  int len_upper;            // upper bound of the length
  int32_t* pinned;          // [4] pinned host words: [0] length, [2] status (1 and 3 unused)
  cudaEvent_t len_event;
  bool len_event_pending;
  int64_t launches;
  int gemm_epoch;           // number of tensor-core projection launches so far (tags the fixup flags)
  // optional per-kernel timing (specasr_profile_*): event pairs recorded around every launch
  bool prof_on;
  std::vector<cudaEvent_t> prof_events;   // 2 per recorded launch
  std::vector<int> prof_kinds;
  size_t prof_used;                       // launches recorded since the last read
  TraceBuf trace;                         // device-side trace, off unless specasr_trace_set was called
  // activation TMA descriptors (tcgen05 path), one per box height 16 << i
  CUtensorMap tm_H[5], tm_AO[5], tm_A[5];
  // tensor-core attention: rotated queries and the two pools
  bool attn_tc;
  CUtensorMap tm_Q, tm_K, tm_V;
};

// Counts a launch and, when profiling is on, brackets it with events on the launching stream.
struct LaunchScope {
  specasr_kv* kv;
  cudaStream_t s;
  LaunchScope(specasr_kv* kv_, int kind, cudaStream_t s_) : kv(kv_), s(s_) {
    kv->launches++;
    if (!kv->prof_on) return;
    if (kv->prof_events.size() < 2 * (kv->prof_used + 1)) {
      cudaEvent_t a, b;
      cudaEventCreate(&a);
      cudaEventCreate(&b);
      kv->prof_events.push_back(a);
      kv->prof_events.push_back(b);
      kv->prof_kinds.push_back(kind);
    }
    kv->prof_kinds[kv->prof_used] = kind;
    cudaEventRecord(kv->prof_events[2 * kv->prof_used], s);
  }
  ~LaunchScope() {
    if (!kv->prof_on) return;
    cudaEventRecord(kv->prof_events[2 * kv->prof_used + 1], s);
    kv->prof_used++;
  }
};

// Launch with programmatic stream serialization: the kernel may start while its predecessor in the
// stream is still running and must call griddepcontrol.wait before it touches anything the predecessor
// writes (every kernel of this library does, whether or not it is launched this way).
template <typename... KArgs, typename... Args>
inline void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Same, for a kernel whose CTAs form clusters of `cluster_x` along x.
template <typename... KArgs, typename... Args>
inline void launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, int cluster_x, cudaStream_t s,
                               Args&&... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = cluster_x;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// One utterance of a (possibly batched) call as the kernels see it: its control block, cache and the workspace
// rows it occupies.  A plain call is one such entry at row 0 of its own workspace.  The table travels as a
// kernel parameter, so the per-utterance kernels (tree prep, embedding, rotary + append, attention, accept) run
// once per call over all utterances.
struct SegDev {
  int32_t* ctl;                 // the utterance's control block
  const int32_t* page_table;
  bf16* k_pool;
  bf16* v_pool;
  const CUtensorMap* tmK;       // device copies of the pool descriptors (tensor-core attention), else null
  const CUtensorMap* tmV;
  int n_pages;
  int row0;                     // first workspace row
  int n;                        // rows
  int chunk;                    // keys per attention CTA
  int capacity;                 // positions the cache can hold
  int pad;
};
struct SegTable {
  int count;
  int splits;                   // grid depth of the attention launch per utterance (largest any of them needs)
  int pad[2];
  SegDev seg[SPECASR_MAX_BATCH];
};

void set_error(const char* fmt, ...);
Workspace carve_workspace(const specasr_model* m, int n_alloc, void* base);
int lm_tiles_of(const specasr_model* m);

// ---- kernels_small.cu
void launch_tree_prep(specasr_kv* wk, const SegTable& t, const int32_t* tokens, const int32_t* parent, cudaStream_t s);
void launch_chain_prep(specasr_kv* kv, int n, bool first, cudaStream_t s);
void launch_embed_tokens(specasr_kv* wk, const SegTable& t, int n_total, const int32_t* tokens, cudaStream_t s);
void launch_copy_embeds(specasr_kv* kv, const float* embeds, int n, cudaStream_t s);
void launch_rmsnorm_split(specasr_kv* wk, const int32_t* ctl, const float* gain, int n, int n_pad, int n_partials,
                          cudaStream_t s);
void launch_rope_append(specasr_kv* wk, const SegTable& t, int n_total, int layer, int n_partials, cudaStream_t s);
void launch_attn_merge(specasr_kv* wk, const int32_t* ctl, int n, int n_pad, int n_splits, cudaStream_t s);
void launch_accept(specasr_kv* wk, const SegTable& t, const int32_t* ctl_shared, const int32_t* tokens,
                   const int32_t* parent, int n_tiles, int32_t* out_argmax, int32_t* out_accept_len, int32_t* out_path,
                   int32_t* out_bonus, cudaStream_t s);
void launch_advance_len(specasr_kv* kv, int n, cudaStream_t s);
void launch_set_len(specasr_kv* kv, int len, cudaStream_t s);
void launch_commit(specasr_kv* kv, const int32_t* path, const int32_t* accept_len, cudaStream_t s);

// ---- attention.cu (plain FMA) / attention_tc.cu (tcgen05)
void launch_tree_attention(specasr_kv* kv, int layer, int n, int n_splits, cudaStream_t s);
bool attention_tc_supported(const specasr_model* m);
bool attention_tc_plan(const specasr_model* m, int n, int total_len, int sm_budget, int max_splits, int* n_splits,
                       int* chunk);
bool attention_tc_make_maps(specasr_kv* kv);
void launch_tree_attention_tc(specasr_kv* wk, const SegTable& t, int n_max, int layer, cudaStream_t s);

// ---- fused_stack.cu: the whole layer stack as one persistent kernel
bool fused_stack_supported(const specasr_kv* wk, int n_total, bool att_tc, int splits);
size_t fused_stack_sync_bytes(const specasr_model* m);
bool launch_fused_stack(specasr_model* m, specasr_kv* wk, const SegTable& tab, int n_total, int n_max,
                        const int32_t* ctl_shared, bool want_head, float* out_logits, bool want_top2, cudaStream_t s);
// top2.cu: top-2 tokens and probabilities of every node from the per-tile pieces the vocabulary epilogue left
void launch_top2_from_tiles(specasr_kv* wk, const SegTable& t, const int32_t* ctl_shared, int n_total, int n_tiles,
                            int32_t* out_ids, float* out_probs, cudaStream_t s);

// ---- gemm_fma.cu / gemm_tcgen05.cu
enum GemmEpilogue {
  EPI_PARTIAL = 0,   // fp32 partial sums [splits][n][M], added up by the consumer kernel
  EPI_SWIGLU = 1,    // SiLU(gate) * up -> hi / lo planes
  EPI_ARGMAX = 2     // per-tile arg-max candidates (+ optional logits)
};
struct GemmArgs {
  const bf16* W;            // [M, K]
  const CUtensorMap* tmW;   // tcgen05 path
  const CUtensorMap* tmAct; // tcgen05 path: activation planes [2 * n_alloc, K]
  const bf16* act;          // [2][n_alloc][K] hi / lo planes
  int M, K, n, n_pad, n_alloc;
  int epilogue;
  int splits;               // EPI_PARTIAL only
  float* P;                 // EPI_PARTIAL: [splits][n_alloc][M]
  bf16* A;                  // EPI_SWIGLU: [2][n_alloc][M/2]
  unsigned long long* amax; // EPI_ARGMAX: [tiles][n_alloc]
  float* logits;            // EPI_ARGMAX: optional [n][M]
  const int32_t* ctl;
};
int gemm_fma_tiles(int M);
void launch_gemm_fma(specasr_kv* kv, const GemmArgs& a, int kind, cudaStream_t s);
int gemm_tc_tiles(int M);
size_t gemm_tc_fixup_bytes(const specasr_model* m, int n_alloc);
int gemm_tc_pick_splits(const specasr_model* m, int M, int K, int n_pad);
void launch_gemm_tc(specasr_kv* kv, const GemmArgs& a, int kind, cudaStream_t s);   // a.ctl = control block to check
bool make_tensor_map_2d(CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer,
                        uint32_t box_inner, uint32_t box_outer);
bool make_act_map(CUtensorMap* out, const void* base, uint64_t K, uint64_t n_alloc, uint32_t box_rows);
// bf16 tensor map of any rank with 128-byte swizzle; strides[i] is the byte stride of dimension i + 1
bool make_tensor_map_nd(CUtensorMap* out, const void* base, int rank, const uint64_t* dims, const uint64_t* strides,
                        const uint32_t* box);
