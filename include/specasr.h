/*
 * specasr.h -- C ABI of the B200 tree-verification library.
 *
 * One verification round of speculative decoding for an LLM-based speech recogniser: the target
 * decoder runs ONE forward pass over a draft token tree on top of a KV cache that already holds the
 * audio-embedding prefix and the text decoded so far, the longest draft path whose tokens equal the
 * target's own greedy tokens is selected, and the accepted nodes' K/V are compacted into contiguous
 * cache slots.  (Draft-then-verify and its lossless property: paper Section II-B; verification of a
 * token tree in one pass with a 2-D attention mask: Section II-B, Fig. 13, and Section IV-C.)
 *
 * Conventions
 *  - Plain C.  No C++ exception crosses this boundary.  Every call returns a specasr_status;
 *    specasr_last_error() gives a thread-local message for the last failure on this thread.
 *  - Pointers marked [device] must be device-accessible on the CUDA device that was current when the
 *    model was created; pointers marked [host] are ordinary host memory.  `stream` is a cudaStream_t
 *    passed as void* (NULL = the legacy default stream).
 *  - Ownership: the caller owns every device buffer (weights, KV pools, page table, workspace,
 *    inputs, outputs).  Handles borrow them and never free them.  The library itself only allocates
 *    the rotary table (device, once per model) and a few bytes of pinned host memory per KV handle.
 *  - Calls are asynchronous on `stream`; outputs are valid once the stream reaches that point.
 *  - Errors that the host can see (null pointer, n out of range, no pending verify, ...) are returned
 *    before anything is enqueued and leave all state untouched.  Errors only the device can see
 *    (malformed parent array, token id out of range, cache capacity exceeded with a length the host
 *    does not know yet, a bounded wait that ran out) set the device status word: the remaining
 *    kernels of that call do nothing, out_accept_len receives -1, and specasr_poll_status reports
 *    the code.  Nothing traps, asserts or spins without a limit.
 *
 * Tree format: tokens[n] and parent_idx[n] with parent_idx[0] = -1 and 0 <= parent_idx[i] < i.
 * Node 0 is the root: the last committed token, whose K/V is not in the cache yet; it is not
 * verified.  Nodes 1..n-1 are draft tokens.  1 <= n <= SPECASR_MAX_NODES.
 */
#ifndef SPECASR_H_
#define SPECASR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPECASR_MAX_NODES 256
#define SPECASR_MAX_BATCH 32

typedef enum specasr_status {
  SPECASR_OK = 0,
  SPECASR_ERR_INVALID_ARG = 1,
  SPECASR_ERR_INVALID_TREE = 2,
  SPECASR_ERR_KV_CAPACITY = 3,
  SPECASR_ERR_STATE = 4,
  SPECASR_ERR_UNSUPPORTED = 5,
  SPECASR_ERR_TIMEOUT = 6,
  SPECASR_ERR_CUDA = 7
} specasr_status;

/* Decoder shape (pre-norm Llama block: RMSNorm, rotary GQA attention, SwiGLU; no biases). */
typedef struct specasr_model_config {
  int32_t n_layers;
  int32_t d_model;
  int32_t n_heads;      /* query heads */
  int32_t n_kv_heads;   /* key/value heads; n_heads % n_kv_heads == 0 */
  int32_t head_dim;     /* 64 or 128 (32 in the cross-check build variant only) */
  int32_t ffn;          /* SwiGLU inner width */
  int32_t vocab;
  int32_t page_size;    /* tokens per KV page; a multiple of 16, at most 208 (16 in the reference workload; any
                           multiple of 8 in the cross-check build variant) */
  int32_t max_positions;/* length of the rotary table = largest position + 1 */
  float rms_eps;
  float rope_base;
  int32_t gemm_path;    /* must be 0: tcgen05 tensor-core projections.  (1 = plain FMA projections exists only in the
                           cross-check build variant of the library, libspecasr_crosscheck.so, which the tests use
                           to compare two engines on a GPU; the product library answers SPECASR_ERR_UNSUPPORTED.) */
  int32_t reserved[3];
} specasr_model_config;

/*
 * Weights, all [device], all borrowed, 16-byte aligned.  Gains are fp32.  The embedding table is bf16, row-major
 * [vocab, d_model] (d_model % 8 == 0).  Every projection matrix W[out_features = M, in_features = K] below (and
 * lm_head) is bf16 and TILE-PACKED: M and K are padded with zeros to multiples of 128, the padded matrix is cut
 * into tiles of 128 rows x 64 columns, every tile is stored contiguously (row-major inside, 16 KB), and the tiles
 * are ordered by row tile, then by column tile.  Element (m, k) therefore sits at element offset
 *   (((m / 128) * Kt + k / 64) * 128 + m % 128) * 64 + k % 64,   Kt = 2 * ceil(K / 128),
 * and the buffer holds ceil(M / 128) * Kt * 8192 elements.  One pipeline stage of a projection (128 rows x 128
 * columns) is then one contiguous 32 KB run of HBM.  The logical row orders of the matrices are:
 *   wqkv[l] : [(n_heads + 2 n_kv_heads) * head_dim, d_model]  rows = all Q heads, all K heads, all V heads;
 *             within every head the rows are in rotary-paired order: stored row 32 g + 16 h + j holds
 *             feature 16 g + j + h * head_dim / 2 (0 <= j < 16, h in {0, 1}), so that a feature and its
 *             rotation partner land in the same warp of the projection's epilogue
 *   wo[l]   : [d_model, n_heads * head_dim]
 *   wgu[l]  : [2 * ffn, d_model]   row 2f = gate row f, row 2f+1 = up row f (interleaved so that one
 *             output tile holds both halves of a SwiGLU feature)
 *   wd[l]   : [d_model, ffn]
 * The per-layer arrays are [host] arrays of n_layers device pointers (copied at create time).
 */
typedef struct specasr_weight_ptrs {
  const void* embed;            /* [vocab, d_model] bf16 */
  const void* lm_head;          /* [vocab, d_model] bf16, tile-packed like the projections */
  const float* g_final;         /* [d_model] */
  const void* const* wqkv;
  const void* const* wo;
  const void* const* wgu;
  const void* const* wd;
  const float* const* g_attn;
  const float* const* g_ffn;
} specasr_weight_ptrs;

typedef struct specasr_model specasr_model;
typedef struct specasr_kv specasr_kv;

/*
 * Handles and bookkeeping (model / workspace / pool sizes / cache handle / length / truncate / status / launch count):
 * no counterpart in the paper, which treats the target decoder as a black box; they exist because a C library needs
 * somewhere to keep the borrowed weight pointers, the tensor maps and the committed length between calls.
 *
 * Creates a model handle on the current CUDA device.  Fails with SPECASR_ERR_UNSUPPORTED for shapes
 * the kernels do not cover (head_dim not 64 or 128, d_model or ffn not a multiple of 8, page_size not a multiple
 * of 16, ...).  Allocates the rotary table and a copy of the weight descriptors on the device, once.
 */
specasr_status specasr_model_create(const specasr_model_config* cfg, const specasr_weight_ptrs* w,
                                    specasr_model** out);
void specasr_model_destroy(specasr_model* m);

/* Bytes of [device] workspace a KV handle needs to verify trees of up to max_nodes nodes.  The library initialises
 * the parts of it that must start in a known state (control words, flags of the projection kernels); the caller
 * need not clear it.  (No counterpart in the paper.) */
size_t specasr_workspace_bytes(const specasr_model* m, int32_t max_nodes);

/* Bytes of ONE of the two KV pools (K and V have the same size) for n_pages pages.
 * Pool layout: [n_layers][n_pages][n_kv_heads][2 planes][page_size][head_dim] bf16; plane 0 is the
 * bf16 rounding of the value, plane 1 the bf16 rounding of the remainder (value ~ hi + lo). */
size_t specasr_kv_pool_bytes(const specasr_model* m, int32_t n_pages);

/*
 * KV handle over caller-owned pools.  page_table [device] int32[max_pages] maps logical page ->
 * physical page (< n_pages); slot s lives in page_table[s / page_size] at offset s % page_size.
 * The capacity is max_pages * page_size slots.  The handle starts empty (length 0).
 * `workspace` [device] of specasr_workspace_bytes(m, max_nodes) bytes, 256-byte aligned.
 */
specasr_status specasr_kv_create(const specasr_model* m, void* k_pool, void* v_pool, int32_t n_pages,
                                 const int32_t* page_table, int32_t max_pages, void* workspace,
                                 int32_t max_nodes, specasr_kv** out);
void specasr_kv_destroy(specasr_kv* kv);

/* Committed length in tokens, [host] out.  If a commit is still in flight the host waits for the event recorded
 * behind it (on the stream that commit was given); `stream` itself is not used.  (No counterpart in the paper.) */
specasr_status specasr_kv_length(specasr_kv* kv, int32_t* out_len, void* stream);
/* Rewinds (or empties) the cache to `len` <= current length.  Drops any pending verify.  Like specasr_kv_length
 * it first waits on the host for a commit in flight (it has to know the current length to check `len`), then
 * enqueues the new length on `stream`.  (No counterpart in the paper.) */
specasr_status specasr_kv_truncate(specasr_kv* kv, int32_t len, void* stream);

/* Context fill (the prefill of Section II-A: audio-embedding vectors followed by prompt text), causal
 * attention, no logits.  embeds [device] fp32 [n, d_model] enter layer 0 directly; tokens [device]
 * int32[n] go through the embedding table.  Any n >= 1 (processed in chunks); advances the length. */
specasr_status specasr_prefill_embeds(specasr_model* m, specasr_kv* kv, const float* embeds, int32_t n, void* stream);
specasr_status specasr_prefill_tokens(specasr_model* m, specasr_kv* kv, const int32_t* tokens, int32_t n, void* stream);

/*
 * Verify a draft token tree (Section II-B; tree mask per Fig. 13 / Section IV-C).
 *   tokens, parent_idx : [device] int32[n_nodes]
 *   out_argmax         : [device] int32[n_nodes]  target greedy token after each node (lowest id on ties)
 *   out_accept_len     : [device] int32[1]        accepted draft nodes on the best path (-1 on device error)
 *   out_path           : [device] int32[n_nodes]  node indices root..best, padded with -1
 * Writes the tree's K/V to cache slots L..L+n-1 (L = committed length) and marks the handle
 * "pending"; the committed length does not change.  Calling verify again without a commit simply
 * overwrites those slots (that is how a round is abandoned).
 */
specasr_status specasr_verify_tree(specasr_model* m, specasr_kv* kv, const int32_t* tokens,
                                   const int32_t* parent_idx, int32_t n_nodes, int32_t* out_argmax,
                                   int32_t* out_accept_len, int32_t* out_path, void* stream);

/* Same, plus optional outputs: out_logits [device] fp32 [n_nodes, vocab] (NULL to skip) and
 * out_bonus [device] int32[1] = out_argmax[best] (the token emitted after the accepted path). */
specasr_status specasr_verify_tree_ex(specasr_model* m, specasr_kv* kv, const int32_t* tokens,
                                      const int32_t* parent_idx, int32_t n_nodes, int32_t* out_argmax,
                                      int32_t* out_accept_len, int32_t* out_path, float* out_logits,
                                      int32_t* out_bonus, void* stream);

/*
 * Verify the draft trees of several utterances in one pass over the weights.  Section II-B defines the
 * verification of one draft (all of its tokens checked by the target model at once); the paper decodes one
 * utterance at a time and has no batched form.  This call applies that same definition to several
 * utterances side by side so that they share one stream of the weights: every utterance keeps its own
 * cache, committed length and tree, and the results are those of `batch` separate specasr_verify_tree calls.
 *   batch              : 1 .. SPECASR_MAX_BATCH
 *   kv                 : [host] `batch` distinct handles of model `m`, all on the tensor-core attention path
 *                        (head_dim 64 or 128, page_size a multiple of 16).  The workspace of kv[0] carries the
 *                        rows of all utterances, so node_offsets[batch] <= max_nodes of kv[0]; it also
 *                        receives the launch counts and profile records of the call.
 *   node_offsets       : [host] int32[batch + 1], node_offsets[0] = 0, strictly increasing; utterance b owns
 *                        nodes node_offsets[b] .. node_offsets[b+1]-1 of the arrays below
 *   tokens, parent_idx : [device] int32[node_offsets[batch]]; parent_idx is local to the utterance
 *                        (-1 for its root, otherwise 0 <= parent < index within the utterance)
 *   out_argmax, out_path : [device] int32[node_offsets[batch]], per utterance as in specasr_verify_tree
 *                        (path entries are local node indices)
 *   out_accept_len     : [device] int32[batch]
 *   out_logits         : [device] fp32 [node_offsets[batch], vocab] or NULL: the target logits after every node
 *   out_bonus          : [device] int32[batch] or NULL
 * Each handle becomes "pending" and is committed on its own:
 *   specasr_commit_kv(m, kv[b], out_path + node_offsets[b], out_accept_len + b, stream).
 * Errors: host-visible ones (null, batch or offsets out of range, a handle twice, a cache that would
 * overflow, SPECASR_ERR_UNSUPPORTED for a handle without the tensor-core attention path) return before
 * anything is enqueued.  A malformed tree fails only its own utterance (its out_accept_len is -1 and its
 * handle's status word is set); a bounded wait that runs out in a kernel shared by all utterances fails
 * every one of them.
 */
specasr_status specasr_verify_tree_batch(specasr_model* m, int32_t batch, specasr_kv* const* kv,
                                         const int32_t* tokens, const int32_t* parent_idx,
                                         const int32_t* node_offsets, int32_t* out_argmax, int32_t* out_accept_len,
                                         int32_t* out_path, float* out_logits, int32_t* out_bonus, void* stream);

/*
 * The same verification with the draft side's quantities computed in the vocabulary projection's epilogue instead of
 * from a materialised logits matrix: for every node the two most probable next tokens and their probabilities under
 * the softmax over the whole vocabulary.  Run on the DRAFT model these are what Section IV reads: drafting stops where
 * the top-1 value falls below a threshold (Section IV-A), and the second-ranked token at such a position seeds a side
 * branch of the sparse tree (Section IV-C).
 *   out_top2_ids   : [device] int32 [n_nodes, 2]  (ties: lower id first; -1 for an utterance whose tree was refused)
 *   out_top2_probs : [device] fp32  [n_nodes, 2]
 * Everything else as in specasr_verify_tree_ex / specasr_verify_tree_batch (no logits output).  Needs the fused layer
 * stack: tensor-core attention (head_dim 64 or 128, page_size a multiple of 16) and at most 64 nodes in the call;
 * otherwise SPECASR_ERR_UNSUPPORTED with nothing enqueued.
 */
specasr_status specasr_verify_tree_top2(specasr_model* m, specasr_kv* kv, const int32_t* tokens,
                                        const int32_t* parent_idx, int32_t n_nodes, int32_t* out_argmax,
                                        int32_t* out_accept_len, int32_t* out_path, int32_t* out_bonus,
                                        int32_t* out_top2_ids, float* out_top2_probs, void* stream);
specasr_status specasr_verify_tree_batch_top2(specasr_model* m, int32_t batch, specasr_kv* const* kv,
                                              const int32_t* tokens, const int32_t* parent_idx,
                                              const int32_t* node_offsets, int32_t* out_argmax,
                                              int32_t* out_accept_len, int32_t* out_path, int32_t* out_bonus,
                                              int32_t* out_top2_ids, float* out_top2_probs, void* stream);

/*
 * Keep the accepted path (after a round control goes back to the draft model, Section II-B, so the cache must
 * hold exactly prefix + accepted tokens): slot L+j <- slot L+path[j] for j = 0..accept_len, all
 * layers, K and V; then L <- L + accept_len + 1.  path / accept_len are the [device] arrays a
 * preceding verify wrote (or the caller's own choice of a root path of that tree).  Requires a
 * pending verify (else SPECASR_ERR_STATE); clears it.  accept_len < 0 on the device (failed verify)
 * makes the commit a no-op.
 */
specasr_status specasr_commit_kv(specasr_model* m, specasr_kv* kv, const int32_t* path,
                                 const int32_t* accept_len, void* stream);

/* Reads the device status word of the last verify/prefill on this handle ([host] out; synchronises
 * `stream`).  SPECASR_OK, SPECASR_ERR_INVALID_TREE, SPECASR_ERR_KV_CAPACITY or SPECASR_ERR_TIMEOUT.
 * (No counterpart in the paper: error reporting of this implementation.) */
specasr_status specasr_poll_status(specasr_kv* kv, int32_t* out_device_status, void* stream);

/* Number of kernels the library has launched on this handle so far (for launch accounting; no counterpart in the
 * paper). */
int64_t specasr_launch_count(const specasr_kv* kv);

/*
 * Optional per-kernel timing for measurement (no counterpart in the paper, which reports only
 * end-to-end latencies, Table 2).  While enabled, every kernel launch on this handle is bracketed by
 * CUDA events on the launching stream.  specasr_profile_read synchronises `stream`, returns the
 * milliseconds and launch counts accumulated per kernel kind since the last read (both [host] arrays
 * of SPECASR_KIND_COUNT entries) and clears them.  Leave it disabled when timing whole calls.
 */
enum {
  SPECASR_KIND_PREP = 0,        /* tree / chain preparation, layer-0 inputs */
  SPECASR_KIND_NORM = 1,        /* RMSNorm + residual + operand split */
  SPECASR_KIND_GEMM_QKV = 2,
  SPECASR_KIND_ROPE = 3,        /* rotary embedding + KV append */
  SPECASR_KIND_ATTN = 4,        /* tree-masked attention */
  SPECASR_KIND_ATTN_MERGE = 5,
  SPECASR_KIND_GEMM_O = 6,
  SPECASR_KIND_GEMM_GU = 7,     /* gate/up projection + SwiGLU */
  SPECASR_KIND_GEMM_DOWN = 8,
  SPECASR_KIND_GEMM_LM = 9,     /* vocabulary projection + argmax */
  SPECASR_KIND_ACCEPT = 10,
  SPECASR_KIND_COMMIT = 11,     /* KV compaction and length bookkeeping */
  SPECASR_KIND_STACK = 12,      /* the whole layer stack (norms, projections, rotary, attention, arg-max) as one
                                   persistent kernel; kinds 1..9 then name its steps in the device-side trace */
  SPECASR_KIND_COUNT = 13
};
specasr_status specasr_profile_enable(specasr_kv* kv, int32_t enable);
/*
 * Device-side trace.  The event pairs of specasr_profile_* sit between launches and thereby switch off the
 * overlap of consecutive kernels (programmatic dependent launch); with a trace buffer set, every thread block of
 * the tree-prep, embedding, norm, projection, rotary, attention, merge and accept kernels instead appends one
 * record of four uint64 words {SPECASR_KIND_*, start, end, wait_end} in %globaltimer nanoseconds (wait_end = when
 * the block's wait for the previous kernel of the stream returned; 0 if it never got there).
 *   buffer : [device] uint64 words, 8-byte aligned: word 0 = number of records appended so far (the caller zeroes it
 *            before a traced call; counting continues past the capacity), word 1 unused, records from word 2 on;
 *            at least 2 + 4 * capacity_records words.  NULL switches tracing off (the default).
 * For a batched call the buffer of the first handle is used.  The buffer is borrowed until it is replaced or the
 * handle is destroyed.  (No counterpart in the paper: instrumentation of this implementation.)
 */
specasr_status specasr_trace_set(specasr_kv* kv, void* buffer, int64_t capacity_records);
specasr_status specasr_profile_read(specasr_kv* kv, double* out_ms, int64_t* out_launches, void* stream);

/*
 * Accept step on its own, for callers that may not allocate.  (The paper has no counterpart: this is a
 * packaging of the accept rule of Section II-B for hosts with a frozen memory plan.)
 *
 * Some users of this library are handed buffers but have no way to get device memory themselves: a
 * plug-in running inside a serving process that reserved all of its device memory at start-up and
 * forbids cudaMalloc afterwards, or a component that scores logits produced elsewhere (another
 * decoder, a replayed trace) and owns nothing but its inputs and outputs.  This call gives them the
 * arg-max + longest-accepted-path step without a model, a KV handle or a workspace.  It calls no
 * cudaMalloc / cudaFree / cudaHostAlloc and no routine that allocates; the only memory it uses besides
 * the arguments is one fixed array of 131328 bytes inside the library image, which every GPU that loads
 * the library holds until the process exits.
 *
 *   logits             : [device] fp32 [n_nodes, vocab], row-major; row i = target logits after node i
 *   tokens, parent_idx : [device] int32[n_nodes], the tree format described at the top of this file
 *   out_argmax         : [device] int32[n_nodes]  arg-max token of every row (lowest id on ties)
 *   out_accept_len     : [device] int32[1]        accepted draft nodes on the best path
 *   out_path           : [device] int32[n_nodes]  node indices root..best, padded with -1
 *   out_bonus          : [device] int32[1] or NULL, out_argmax[best]
 * Same rule and same tie-breaks as specasr_verify_tree, so feeding it the logits of
 * specasr_verify_tree_ex reproduces that call's out_argmax / out_accept_len / out_path / out_bonus.
 *
 * Limits and errors: 1 <= n_nodes <= SPECASR_MAX_NODES (the fixed array has room for exactly that many
 * nodes; larger trees are refused with SPECASR_ERR_INVALID_ARG and a message that says so), vocab >= 1.
 * A malformed parent array or a token id outside [0, vocab) is found on the device: out_accept_len
 * receives -1 and out_argmax / out_path are filled with -1.
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that
 * device current); make that first call outside any stream capture.  Asynchronous on `stream`.
 * All calls on one device share the array, and it keeps what the last call left in it (the call clears
 * the part that has to start at zero): two calls that overlap on the GPU, e.g. on different streams,
 * race on it and may both return wrong results.  Issue them on one stream or order them with events.
 */
specasr_status specasr_accept_logits_static(const float* logits, int32_t vocab, const int32_t* tokens,
                                            const int32_t* parent_idx, int32_t n_nodes, int32_t* out_argmax,
                                            int32_t* out_accept_len, int32_t* out_path, int32_t* out_bonus,
                                            void* stream);

/*
 * Top-2 tokens and their probabilities for every row of a logits matrix (the draft side of the method:
 * Section IV-A truncates a draft where the normalised value of its top-1 token falls below a threshold,
 * Section IV-C branches on the second-ranked token there).
 *   logits    : [device] fp32 [n_rows, vocab], row-major, finite values (e.g. out_logits of
 *               specasr_verify_tree_ex run on the draft model)
 *   out_ids   : [device] int32 [n_rows, 2]  most probable and second most probable token (ties: lower id first;
 *               both entries equal when vocab == 1)
 *   out_probs : [device] fp32 [n_rows, 2]   their probabilities under the softmax over the whole row
 * No scratch memory; one kernel on `stream`.  Errors: null pointer, n_rows < 1, vocab < 1 ->
 * SPECASR_ERR_INVALID_ARG with nothing enqueued.
 */
specasr_status specasr_top2_probs(const float* logits, int32_t n_rows, int32_t vocab, int32_t* out_ids,
                                  float* out_probs, void* stream);

const char* specasr_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SPECASR_H_ */
