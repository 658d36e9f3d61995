// cast_accept (target argmax sweep + greedy walk) and cast_compact_kv.
#include <math.h>

#include "cast_internal.h"

using namespace cast;

namespace {

template <typename T> struct Vec;
template <> struct Vec<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void load(const float* p, float* out) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(p));
    out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
  }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float* out) {
    const uint4 a = __ldcs(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      out[2 * i] = __uint_as_float(w[i] << 16);
      out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};

constexpr int kArgThreads = 256;
constexpr int kArgUnroll = 8;

// One CTA per (chunk, tree token, sequence): the largest (logit, lowest token id) of the chunk. (Consecutive CTAs
// sweep consecutive memory; with the token index slowest, so that the rows past the trees come last, the large
// batches lost a sixth of their bandwidth.)
template <typename T>
__global__ void __launch_bounds__(kArgThreads) argmax_sweep_kernel(const T* __restrict__ logits, int V, int Ncap,
                                                                   int chunk_elems, const int32_t* __restrict__ n_tree,
                                                                   unsigned long long* __restrict__ part) {
  __shared__ unsigned long long red[kArgThreads / 32];
  const int chunk = blockIdx.x, t = blockIdx.y, b = blockIdx.z;
  // the walk kernel that follows may become resident now (it waits for this grid before it reads the winners)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (t >= n_tree[b]) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t row = (size_t)b * Ncap + t;
  const T* x = logits + row * V;
  const int begin = chunk * chunk_elems;
  const int end = min(begin + chunk_elems, V);
  constexpr int VEC = Vec<T>::N;
  const bool aligned = (reinterpret_cast<uintptr_t>(x) & 15) == 0;
  float best = -INFINITY;
  int barg = -1;
  for (int base = begin; base < end; base += kArgThreads * VEC * kArgUnroll) {
    float xv[kArgUnroll * VEC];
#pragma unroll
    for (int v = 0; v < kArgUnroll; ++v) {
      const int idx = base + (v * kArgThreads + tid) * VEC;
      if (aligned && idx + VEC <= end) {
        Vec<T>::load(x + idx, xv + v * VEC);
      } else {
#pragma unroll
        for (int e = 0; e < VEC; ++e) xv[v * VEC + e] = (idx + e < end) ? to_float(x[idx + e]) : -INFINITY;
      }
    }
#pragma unroll
    for (int i = 0; i < kArgUnroll * VEC; ++i)
      if (xv[i] > best) {  // ids ascend within a thread: the first maximum has the lowest id
        best = xv[i];
        barg = base + ((i / VEC) * kArgThreads + tid) * VEC + (i % VEC);
      }
  }
  unsigned long long key = barg >= 0 ? make_key(best, barg) : 0ull;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
    key = other > key ? other : key;
  }
  if (lane == 0) red[warp] = key;
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kArgThreads / 32; ++w) key = red[w] > key ? red[w] : key;
    part[row * kAcceptMaxChunks + chunk] = key;
  }
}

// One CTA per sequence: merge the chunk winners into g[t], then walk from the root.
__global__ void __launch_bounds__(CAST_MAX_TREE) accept_walk_kernel(
    const unsigned long long* __restrict__ part, int nchunks, int Ncap, int Nmax, int H, const int32_t* __restrict__ tokens,
    const int32_t* __restrict__ parent, const int32_t* __restrict__ n_tree, int32_t* __restrict__ accept_len,
    int32_t* __restrict__ accept_path, int32_t* __restrict__ bonus, DevState* st) {
  __shared__ int g[CAST_MAX_TREE], tok[CAST_MAX_TREE], par[CAST_MAX_TREE];
  const int b = blockIdx.x, t = threadIdx.x, lane = t & 31;
  int N = n_tree[b];
  if (N > Nmax) N = 0;  // rows past Nmax were not swept: refused like an empty tree
  if (N < 1) {
    if (t == 0) {
      report(st, CAST_ERR_BAD_TREE, b);
      accept_len[b] = 0;
      bonus[b] = 0;
      for (int j = 0; j <= H; ++j) accept_path[b * (H + 1) + j] = -1;
    }
    return;
  }
  // the tree arrays were written before the sweep was launched; the sweep's winners are read after the wait
  // (programmatic dependent launch: this grid may be resident while the sweep still runs; a no-op otherwise)
  int tok_mine = 0, par_mine = -1;
  if (t < N) {
    tok_mine = tokens[(size_t)b * Ncap + t];
    par_mine = parent[(size_t)b * Ncap + t];
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (t < N) {
    unsigned long long key = 0ull;
    for (int c = 0; c < nchunks; ++c) {
      const unsigned long long k = part[((size_t)b * Ncap + t) * kAcceptMaxChunks + c];
      key = k > key ? k : key;
    }
    g[t] = key ? key_token(key) : 0;
    tok[t] = tok_mine;
    par[t] = par_mine;
    if ((t == 0 && par[t] != -1) || (t > 0 && (par[t] < 0 || par[t] >= t))) report(st, CAST_ERR_BAD_TREE, b * Ncap + t);
  }
  __syncthreads();
  if (t >= 32) return;
  int cur = 0, len = 0;
  if (lane == 0) accept_path[b * (H + 1)] = 0;
  while (true) {
    const int want = g[cur];
    int found = 0x7fffffff;
    for (int c = lane; c < N; c += 32)
      if (par[c] == cur && tok[c] == want) {
        found = c;
        break;
      }
    found = __reduce_min_sync(0xffffffffu, found);
    if (found == 0x7fffffff) break;
    if (len == H || found <= cur) {  // deeper than the path buffer, or not a forward edge
      if (lane == 0) report(st, CAST_ERR_BAD_TREE, b * Ncap + found);
      break;
    }
    cur = found;
    ++len;
    if (lane == 0) accept_path[b * (H + 1) + len] = cur;
  }
  if (lane == 0) {
    for (int j = len + 1; j <= H; ++j) accept_path[b * (H + 1) + j] = -1;
    accept_len[b] = len;
    bonus[b] = g[cur];
  }
}

// ------------------------------------------------------------------ compaction
constexpr int kCompactThreads = 256;
constexpr int kCompactItems = 8;  // 16-byte pieces per thread

struct CompactParams {
  char* k;
  char* v;
  size_t layer_stride;
  int Hkv, row_bytes, page_size, seq_capacity, num_pages, H1;
  const int32_t* page_table;
  const int32_t* accept_path;
  const int32_t* accept_len;
  int32_t* kv_len;
  int32_t* ticket;
  DevState* st;
};

__device__ __forceinline__ size_t cache_row_offset(const CompactParams& p, int b, int pos, int h, bool* bad) {
  size_t slot;
  if (p.page_size == 0) {
    slot = (size_t)b * p.seq_capacity + pos;
  } else {
    const int page = p.page_table[(size_t)b * p.seq_capacity + pos / p.page_size];
    if (page < 0 || page >= p.num_pages) {
      *bad = true;
      return 0;
    }
    slot = (size_t)page * p.page_size + pos % p.page_size;
  }
  return (slot * p.Hkv + h) * (size_t)p.row_bytes;
}

// One CTA per (kv-head, layer, sequence). Every source row is in registers before the first
// store, so a destination slot that is also a later source (path 0,2,3: slot 2) is safe.
__global__ void __launch_bounds__(kCompactThreads) compact_kernel(const CompactParams p) {
  const int h = blockIdx.x, layer = blockIdx.y, b = blockIdx.z, tid = threadIdx.x;
  const int L = p.kv_len[b];
  int a = p.accept_len[b];
  if (a < 0) a = 0;
  if (a > p.H1 - 1) a = p.H1 - 1;
  const int rows = a + 1, vpr = p.row_bytes / 16;
  const int per = rows * vpr, items = 2 * per;
  const int max_pos = p.page_size == 0 ? p.seq_capacity : p.seq_capacity * p.page_size;
  uint4 buf[kCompactItems];
  bool bad = false;
#pragma unroll
  for (int it = 0; it < kCompactItems; ++it) {
    const int i = it * kCompactThreads + tid;
    if (i < items) {
      const int which = i / per, rem = i % per, j = rem / vpr, vv = rem % vpr;
      const int src = p.accept_path[b * p.H1 + j];
      const int pos = L + src;
      // a path element is a tree index no smaller than its place on the path (parents precede children), so
      // the destination L + j never lies past the source; anything else is a malformed path
      if (L < 0 || src < j || pos >= max_pos) {
        bad = true;
        continue;
      }
      const size_t off = cache_row_offset(p, b, pos, h, &bad);
      char* base = (which ? p.v : p.k) + (size_t)layer * p.layer_stride;
      if (!bad) buf[it] = *reinterpret_cast<const uint4*>(base + off + (size_t)vv * 16);
    }
  }
  const int any_bad = __syncthreads_or(bad ? 1 : 0);
  if (any_bad) {
    if (tid == 0) report(p.st, CAST_ERR_BAD_PAGE, b);
  } else {
#pragma unroll
    for (int it = 0; it < kCompactItems; ++it) {
      const int i = it * kCompactThreads + tid;
      if (i < items) {
        const int which = i / per, rem = i % per, j = rem / vpr, vv = rem % vpr;
        bool bad2 = false;
        const size_t off = cache_row_offset(p, b, L + j, h, &bad2);
        char* base = (which ? p.v : p.k) + (size_t)layer * p.layer_stride;
        if (!bad2) *reinterpret_cast<uint4*>(base + off + (size_t)vv * 16) = buf[it];
      }
    }
  }
  // the last CTA of the sequence (every CTA has read kv_len[b] by then) publishes the new length
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    const int t = atomicAdd(&p.ticket[b], 1);
    if (t == (int)(gridDim.x * gridDim.y) - 1) {
      p.ticket[b] = 0;
      if (!any_bad) p.kv_len[b] = L + a + 1;
    }
  }
}

}  // namespace

extern "C" cast_status cast_accept(cast_ctx* c, const void* target_logits, cast_dtype dtype, int B,
                                   const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                   const uint32_t* anc_mask, const int32_t* n_tree, int32_t* accept_len,
                                   int32_t* accept_path, int32_t* bonus_token, void* stream) {
  (void)depth;
  (void)anc_mask;
  if (!c || !target_logits || !tokens || !parent || !n_tree || !accept_len || !accept_path || !bonus_token || B < 1)
    return CAST_ERR_INVALID_ARG;
  if (dtype != CAST_F32 && dtype != CAST_BF16) return CAST_ERR_DTYPE;
  if (B > c->cfg.max_batch) return CAST_ERR_CAPACITY;
  const int V = c->cfg.vocab, Ncap = c->cfg.max_tree;
  // Chunks per logits row: enough CTAs to keep four per SM streaming when every sequence verifies its full
  // budget (the context's total_token; the row slots beyond a tree exit at once), and never chunks of more
  // than 32 K logits, so that a batch whose trees came out far below the budget still has several live CTAs
  // per SM; at least 4096 logits per chunk.
  const int budget = c->cfg.total_token < Ncap ? c->cfg.total_token : Ncap;
  int nchunks = (4 * c->num_sms + B * budget - 1) / (B * budget);
  if (nchunks < (V + 32767) / 32768) nchunks = (V + 32767) / 32768;
  if (nchunks > kAcceptMaxChunks) nchunks = kAcceptMaxChunks;
  if (nchunks > V / 4096) nchunks = V / 4096;
  if (nchunks < 1) nchunks = 1;
  // A CTA sweeps its chunk in rounds of kArgThreads * kArgUnroll vectors, each a full memory latency whether
  // the round is full or not: among the counts within two of the one above, the one whose last round is
  // fullest (V = 128 256 fp32 at batch 1: 8 chunks of 1.96 rounds instead of 10 of 1.57, 10.3 -> 9.4 us).
  {
    const int round_elems = kArgThreads * kArgUnroll * (dtype == CAST_F32 ? 4 : 8);
    const int lo = (V + 32767) / 32768 > nchunks - 2 ? (V + 32767) / 32768 : nchunks - 2;
    int hi = nchunks + 2 < kAcceptMaxChunks ? nchunks + 2 : kAcceptMaxChunks;
    if (hi > V / 4096) hi = V / 4096;
    const int n0 = nchunks;
    long long best = -1;
    for (int n = lo < 1 ? 1 : lo; n <= hi; ++n) {
      const int ce = ((V + n - 1) / n + 7) / 8 * 8;
      const long long padded = (long long)((ce + round_elems - 1) / round_elems) * round_elems * n;  // logits' worth of rounds
      const int dist = n > n0 ? n - n0 : n0 - n, dist_best = nchunks > n0 ? nchunks - n0 : n0 - nchunks;
      if (best < 0 || padded < best || (padded == best && dist <= dist_best)) {  // ties: nearest to n0, the larger of two
        best = padded;
        nchunks = n;
      }
    }
  }
  int chunk_elems = (V + nchunks - 1) / nchunks;
  chunk_elems = (chunk_elems + 7) / 8 * 8;
  nchunks = (V + chunk_elems - 1) / chunk_elems;
  cudaStream_t s = (cudaStream_t)stream;
  const dim3 grid(nchunks, budget, B);  // rows a tree of this context can have; a larger n_tree is BAD_TREE
  if (dtype == CAST_F32)
    argmax_sweep_kernel<float><<<grid, kArgThreads, 0, s>>>((const float*)target_logits, V, Ncap, chunk_elems, n_tree,
                                                            c->acc_part);
  else
    argmax_sweep_kernel<__nv_bfloat16><<<grid, kArgThreads, 0, s>>>((const __nv_bfloat16*)target_logits, V, Ncap,
                                                                    chunk_elems, n_tree, c->acc_part);
  {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(B, 1, 1);
    cfg.blockDim = dim3(CAST_MAX_TREE, 1, 1);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // resident while the sweep drains
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const unsigned long long* part = c->acc_part;
    const int H = c->cfg.max_depth;
    DevState* st = c->state;
    if (cudaLaunchKernelEx(&cfg, accept_walk_kernel, part, nchunks, Ncap, budget, H, tokens, parent, n_tree, accept_len,
                           accept_path, bonus_token, st) != cudaSuccess) {
      cudaGetLastError();
      return CAST_ERR_CUDA;
    }
  }
  return launch_status();
}

// ---- cast_accept_static: the acceptance step for callers that must not allocate ----------------
// Scratch for the chunk winners of the target argmax sweep. It lives in the library image: every GPU
// that loads the library holds these 512 KB until the process exits.
constexpr int kStaticAcceptRows = 2048;  // B * Ncap at most
static __device__ __align__(256) unsigned long long g_accept_static_scratch[kStaticAcceptRows * kAcceptMaxChunks];
// The walk kernel records a malformed tree in a state block. Without a context there is none, so the
// record goes to this one, which nobody reads (first record sticks; it never needs clearing).
static __device__ __align__(256) cast::DevState g_accept_static_sink;

namespace {
// Device address of the scratch array, looked up once per device. In host code the array's name is
// only a stand-in for the symbol; the address a kernel can use comes from cudaGetSymbolAddress.
cast_status static_scratch_address(unsigned long long** out, DevState** sink) {
  constexpr int kMaxDevices = 64;
  static unsigned long long* addr[kMaxDevices] = {nullptr};
  static DevState* sink_addr[kMaxDevices] = {nullptr};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CAST_ERR_CUDA;
  if (addr[dev] == nullptr || sink_addr[dev] == nullptr) {
    void* p = nullptr;
    void* q = nullptr;
    if (cudaGetSymbolAddress(&p, g_accept_static_scratch) != cudaSuccess || p == nullptr) return CAST_ERR_CUDA;
    if (cudaGetSymbolAddress(&q, g_accept_static_sink) != cudaSuccess || q == nullptr) return CAST_ERR_CUDA;
    addr[dev] = static_cast<unsigned long long*>(p);
    sink_addr[dev] = static_cast<DevState*>(q);
  }
  *out = addr[dev];
  *sink = sink_addr[dev];
  return CAST_OK;
}
}  // namespace

extern "C" cast_status cast_accept_static(const void* target_logits, cast_dtype dtype, int B, int n_cap, int vocab,
                                          int max_depth, const int32_t* tokens, const int32_t* parent,
                                          const int32_t* n_tree, int32_t* accept_len, int32_t* accept_path,
                                          int32_t* bonus_token, void* stream) {
  if (!target_logits || !tokens || !parent || !n_tree || !accept_len || !accept_path || !bonus_token || B < 1 ||
      n_cap < 1 || vocab < 1 || max_depth < 1)
    return CAST_ERR_INVALID_ARG;
  if (dtype != CAST_F32 && dtype != CAST_BF16) return CAST_ERR_DTYPE;
  if (n_cap > CAST_MAX_TREE || max_depth > CAST_MAX_DEPTH || (long long)B * n_cap > kStaticAcceptRows)
    return CAST_ERR_CAPACITY;
  unsigned long long* scratch = nullptr;
  DevState* sink = nullptr;
  const cast_status st = static_scratch_address(&scratch, &sink);
  if (st != CAST_OK) return st;
  int num_sms = 0, dev = 0;
  CAST_CUDA_OK(cudaGetDevice(&dev));
  CAST_CUDA_OK(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev));
  int nchunks = (4 * num_sms + B * n_cap - 1) / (B * n_cap);
  if (nchunks > kAcceptMaxChunks) nchunks = kAcceptMaxChunks;
  if (nchunks > vocab / 4096) nchunks = vocab / 4096;
  if (nchunks < 1) nchunks = 1;
  int chunk_elems = (vocab + nchunks - 1) / nchunks;
  chunk_elems = (chunk_elems + 7) / 8 * 8;
  nchunks = (vocab + chunk_elems - 1) / chunk_elems;
  cudaStream_t s = (cudaStream_t)stream;
  const dim3 grid(nchunks, n_cap, B);
  // every chunk winner that the walk reads is written by this call's sweep first: nothing to clear
  if (dtype == CAST_F32)
    argmax_sweep_kernel<float><<<grid, kArgThreads, 0, s>>>((const float*)target_logits, vocab, n_cap, chunk_elems,
                                                            n_tree, scratch);
  else
    argmax_sweep_kernel<__nv_bfloat16><<<grid, kArgThreads, 0, s>>>((const __nv_bfloat16*)target_logits, vocab, n_cap,
                                                                    chunk_elems, n_tree, scratch);
  accept_walk_kernel<<<B, CAST_MAX_TREE, 0, s>>>(scratch, nchunks, n_cap, n_cap, max_depth, tokens, parent, n_tree, accept_len,
                                                 accept_path, bonus_token, sink);
  return launch_status();
}

extern "C" cast_status cast_compact_kv(cast_ctx* c, void* k_cache, void* v_cache, cast_dtype dtype, int B,
                                       int n_layers, size_t layer_stride_bytes, int Hkv, int D, int page_size,
                                       const int32_t* page_table, int seq_capacity, int num_pages,
                                       const int32_t* accept_path, const int32_t* accept_len, int32_t* kv_len,
                                       void* stream) {
  if (!c || !k_cache || !v_cache || !accept_path || !accept_len || !kv_len || B < 1 || n_layers < 1 || Hkv < 1 ||
      D < 1 || page_size < 0 || seq_capacity < 1 || (page_size > 0 && (!page_table || num_pages < 1)))
    return CAST_ERR_INVALID_ARG;
  if (dtype != CAST_F32 && dtype != CAST_BF16) return CAST_ERR_DTYPE;
  if (B > c->cfg.max_batch) return CAST_ERR_CAPACITY;
  const int row_bytes = D * (dtype == CAST_F32 ? 4 : 2);
  if (row_bytes % 16 != 0) return CAST_ERR_SHAPE;
  if (((uintptr_t)k_cache | (uintptr_t)v_cache | layer_stride_bytes) & 15) return CAST_ERR_SHAPE;
  const int H1 = c->cfg.max_depth + 1;
  if (2 * H1 * (row_bytes / 16) > kCompactThreads * kCompactItems) return CAST_ERR_CAPACITY;
  c->tree_inputs_fresh = 1;  // kv_len and cache rows: an attention call that follows reads them after its dependency wait
  CompactParams p;
  p.k = (char*)k_cache; p.v = (char*)v_cache; p.layer_stride = layer_stride_bytes;
  p.Hkv = Hkv; p.row_bytes = row_bytes; p.page_size = page_size; p.seq_capacity = seq_capacity;
  p.num_pages = num_pages; p.H1 = H1;
  p.page_table = page_table; p.accept_path = accept_path; p.accept_len = accept_len; p.kv_len = kv_len;
  p.ticket = c->compact_ticket; p.st = c->state;
  compact_kernel<<<dim3(Hkv, n_layers, B), kCompactThreads, 0, (cudaStream_t)stream>>>(p);
  return launch_status();
}
