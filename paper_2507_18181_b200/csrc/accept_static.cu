// specasr_accept_logits_static: greedy acceptance over a draft token tree from a caller-supplied logits
// matrix, using no memory beyond the caller's buffers and one fixed array that lives inside this
// library.  See include/specasr.h for the contract.
//
// Two kernels.  k_logit_keys_static scans the vocabulary in kStaticChunks slices per node and leaves one
// packed (ordered logit, ~token id) candidate per slice in the fixed array; k_accept_static checks the
// parent array, reduces the candidates to the arg-max token of every node (lowest id on ties) and walks
// the tree exactly like the accept step of specasr_verify_tree: a draft node is kept while its token
// equals the arg-max at its parent, the deepest kept node (lowest index among equals) wins.
#include <mutex>

#include "internal.h"
#include "device_utils.cuh"

namespace {

constexpr int kStaticChunks = 64;                                     // vocabulary slices per node
constexpr int kStaticCtlBytes = 256;                                  // word 0: device status of the last call
constexpr size_t kStaticKeyBytes = (size_t)kStaticChunks * SPECASR_MAX_NODES * sizeof(unsigned long long);
constexpr size_t kStaticBytes = kStaticCtlBytes + kStaticKeyBytes;    // 131328 bytes held by every device that loads the library

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress, never an address
// a kernel could use; device code below receives the real address as an argument.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices];     // device address of g_static_scratch, per device, filled on first use

__global__ void __launch_bounds__(256) k_logit_keys_static(const float* __restrict__ logits, int vocab, int n,
                                                           unsigned long long* __restrict__ keys) {
  __shared__ unsigned long long s_best[8];
  const int node = blockIdx.y, chunk = blockIdx.x;
  const long long v0 = (long long)chunk * vocab / kStaticChunks, v1 = (long long)(chunk + 1) * vocab / kStaticChunks;
  const float* row = logits + (size_t)node * vocab;
  unsigned long long best = 0ull;
  for (long long v = v0 + threadIdx.x; v < v1; v += 256) {
    const unsigned long long key = pack_max_key(row[v], (uint32_t)v);
    best = key > best ? key : best;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, best, o);
    best = other > best ? other : best;
  }
  if ((threadIdx.x & 31) == 0) s_best[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) best = s_best[w] > best ? s_best[w] : best;
    keys[(size_t)chunk * SPECASR_MAX_NODES + node] = best;      // 0 = empty slice (vocab < kStaticChunks)
  }
  (void)n;
}

__global__ void __launch_bounds__(256) k_accept_static(int32_t* __restrict__ status,
                                                       const unsigned long long* __restrict__ keys,
                                                       const int32_t* __restrict__ tokens,
                                                       const int32_t* __restrict__ parent, int n, int vocab,
                                                       int32_t* __restrict__ out_argmax,
                                                       int32_t* __restrict__ out_accept_len,
                                                       int32_t* __restrict__ out_path, int32_t* __restrict__ out_bonus) {
  __shared__ int s_arg[SPECASR_MAX_NODES];
  __shared__ int s_depth[SPECASR_MAX_NODES];
  __shared__ unsigned int s_best;
  __shared__ int s_bad;
  const int i = threadIdx.x;
  if (i == 0) {
    s_bad = 0;
    s_best = 0u;
  }
  __syncthreads();
  if (i < n) {
    const int p = parent[i], t = tokens[i];
    if ((i == 0 ? p != -1 : (p < 0 || p >= i)) || t < 0 || t >= vocab) atomicOr(&s_bad, 1);
  }
  __syncthreads();
  if (s_bad) {
    if (i < n) {
      out_argmax[i] = -1;
      out_path[i] = -1;
    }
    if (i == 0) {
      status[0] = SPECASR_ERR_INVALID_TREE;
      out_accept_len[0] = -1;
      if (out_bonus) out_bonus[0] = -1;
    }
    return;
  }
  if (i < n) {
    unsigned long long best = 0ull;
    for (int c = 0; c < kStaticChunks; ++c) {
      const unsigned long long v = keys[(size_t)c * SPECASR_MAX_NODES + i];
      best = v > best ? v : best;
    }
    const int tok = (int)(0xFFFFFFFFu - (unsigned int)(best & 0xFFFFFFFFull));
    s_arg[i] = tok;
    out_argmax[i] = tok;
    out_path[i] = -1;
    int d = 0;
    for (int j = i; j > 0 && d <= n; j = parent[j]) ++d;     // parent[j] < j was checked: the walk ends
    s_depth[i] = d;
  }
  __syncthreads();
  if (i < n) {
    bool ok = true;
    int steps = 0;
    for (int j = i; j > 0 && steps <= n; ++steps) {
      const int p = parent[j];
      ok = ok && (tokens[j] == s_arg[p]);
      j = p;
    }
    if (ok) atomicMax(&s_best, ((unsigned int)s_depth[i] << 16) | (unsigned int)(0xFFFF - i));
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

}  // namespace

extern "C" specasr_status specasr_accept_logits_static(const float* logits, int32_t vocab, const int32_t* tokens,
                                                       const int32_t* parent_idx, int32_t n_nodes,
                                                       int32_t* out_argmax, int32_t* out_accept_len,
                                                       int32_t* out_path, int32_t* out_bonus, void* stream) {
  if (!logits || !tokens || !parent_idx || !out_argmax || !out_accept_len || !out_path) {
    set_error("specasr_accept_logits_static: null argument");
    return SPECASR_ERR_INVALID_ARG;
  }
  if (n_nodes < 1 || n_nodes > SPECASR_MAX_NODES) {
    set_error("specasr_accept_logits_static: n_nodes = %d exceeds what the built-in scratch array holds (1..%d nodes)",
              n_nodes, SPECASR_MAX_NODES);
    return SPECASR_ERR_INVALID_ARG;
  }
  if (vocab < 1) {
    set_error("specasr_accept_logits_static: vocab must be >= 1");
    return SPECASR_ERR_INVALID_ARG;
  }
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    set_error("specasr_accept_logits_static: no current CUDA device below index %d (%s)", kMaxDevices,
              cudaGetErrorString(e));
    return SPECASR_ERR_CUDA;
  }
  void* base = nullptr;
  {
    // first call on this device: look up where the device keeps the array (no allocation happens here)
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
      void* p = nullptr;
      e = cudaGetSymbolAddress(&p, g_static_scratch);
      if (e != cudaSuccess || !p) {
        set_error("specasr_accept_logits_static: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
        return SPECASR_ERR_CUDA;
      }
      g_static_ptr[dev] = p;
    }
    base = g_static_ptr[dev];
  }
  cudaStream_t s = (cudaStream_t)stream;
  int32_t* status = (int32_t*)base;
  unsigned long long* keys = (unsigned long long*)((unsigned char*)base + kStaticCtlBytes);
  // the array keeps whatever the previous call left: the status word must start at zero; the key slots
  // of nodes 0..n-1 are all rewritten by the first kernel, the others are never read
  e = cudaMemsetAsync(status, 0, kStaticCtlBytes, s);
  if (e != cudaSuccess) {
    set_error("specasr_accept_logits_static: cudaMemsetAsync failed: %s", cudaGetErrorString(e));
    return SPECASR_ERR_CUDA;
  }
  k_logit_keys_static<<<dim3(kStaticChunks, n_nodes), 256, 0, s>>>(logits, vocab, n_nodes, keys);
  k_accept_static<<<1, 256, 0, s>>>(status, keys, tokens, parent_idx, n_nodes, vocab, out_argmax, out_accept_len,
                                    out_path, out_bonus);
  e = cudaGetLastError();
  if (e != cudaSuccess) {
    set_error("specasr_accept_logits_static: launch failed: %s", cudaGetErrorString(e));
    return SPECASR_ERR_CUDA;
  }
  return SPECASR_OK;
}
