// Internal declarations shared by the CUDA translation units of the CAST library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <map>

#include "cast.h"

namespace cast {

// ---- device-resident per-step state ---------------------------------------
struct DevState {
  int32_t B;
  int32_t pad0;
  int32_t pool_size;    // nodes per sequence so far (root included)
  int32_t ctx_sum;      // sum_{j=1}^{i-1} n_j  (context of Eq. 2)
  int32_t n0;           // padded context length = max_b kv_len[b]
  int32_t layers_done;
  int32_t n_tree;       // N of the last rerank
  int32_t kept_total;   // 1 + sum n_j (pool size in pool_mode 1)
  double u_last;        // u^{(i)}_{n_i} of the last generated layer
  int32_t n_hist[CAST_MAX_DEPTH + 1];
  // rows[i]: logits rows that expand call i reads (n_{i-1}; 0: expansion is over). Layer i's
  // kernel only reads rows[i] and writes rows[i+1], so CTAs that start late see a stable value.
  int32_t rows[CAST_MAX_DEPTH + 2];
  // layer i's candidates sit at pool positions [layer_base[i], layer_base[i] + layer_n[i])
  int32_t layer_base[CAST_MAX_DEPTH + 1];
  int32_t layer_n[CAST_MAX_DEPTH + 1];
  int32_t status[2];    // first device-detected error and its detail
};

struct DevTable {  // S_T(B), S_D(B) on the device
  int32_t L, M, Ntab;
  const double* fT;  // [M][Ntab]
  const double* fD;  // [M][Ntab]
};

struct HostTable {
  DevTable dev;
  double* storage;  // one allocation: fT then fD
};

// Limits of the vocabulary sweep.
constexpr int kSweepThreads = 512;
constexpr int kSweepEpt = 32;                             // logits per thread per pass
constexpr int kSweepSub = kSweepThreads * kSweepEpt;      // logits per CTA per pass
constexpr int kSweepMaxChunks = 8;                        // CTAs per logits row: one thread-block cluster
constexpr int kCandCap = 4096;                            // 64-bit keys of shared scratch per CTA (warp lists, short list)
constexpr int kMaxFifo = 64;
constexpr int kAcceptMaxChunks = 32;
constexpr int kAttnWorkListCap = 4096;                    // CTAs of an attention launch that a work list can describe

}  // namespace cast

struct cast_ctx {
  cast_config cfg;
  int W;          // effective width
  int P;          // pool capacity per sequence
  int words;      // mask words per tree token
  int device;
  int num_sms;

  // pool, structure of arrays [max_batch][P]
  double* pool_score;
  int32_t* pool_token;
  int32_t* pool_parent;
  int32_t* pool_depth;
  uint8_t* pool_kept;
  int32_t* retained;   // [max_batch][W] pool indices of the last layer's retained nodes
  // every layer's candidates in descending order: pool index and log-value at position base + rank
  int32_t* lsort;      // [max_batch][P]
  double* lscore;      // [max_batch][P]

  cast::DevState* state;

  // what the step's first expand call reads (set by cast_step_begin)
  const int32_t* step_root;
  const int32_t* step_kv_len;

  int32_t* layer_ticket;          // [1]
  // batched layer tail: per-sequence tickets and what every sequence hands to the batch-wide part
  int32_t* seq_ticket;            // [max_batch]
  double* tail_vs;                // [max_batch][CAST_MAX_WIDTH] values of the first n sorted candidates
  int32_t* tail_sorted;           // [max_batch][CAST_MAX_WIDTH] their pool indices
  int32_t* tail_tok;              // [max_batch][CAST_MAX_WIDTH] their tokens

  // depth-pruning buffers
  double* fifo_vals;   // [H-1][R]
  int32_t* fifo_cnt;   // [H-1]

  // rerank scratch
  double* sel_score;   // [max_batch][Ncap]
  double* sel_value;   // [max_batch][Ncap]
  int32_t* sel_idx;    // [max_batch][Ncap]

  // acceptance scratch
  unsigned long long* acc_part;  // [max_batch*Ncap][kAcceptMaxChunks]
  int32_t* compact_ticket;       // [max_batch]

  // attention workspace (grown on demand)
  void* attn_ws;
  size_t attn_ws_bytes;
  // workspace of the tensor-core attention's global-merge mode: tickets, then split partials
  void* attn_tc_ws;
  size_t attn_tc_ws_bytes;

  // stochastic acceptance, per logits dtype (0 fp32, 1 bf16): cluster size found to be launchable
  // (0: not looked up yet) and whether a CTA's vocabulary slice is cached in shared memory
  int sto_cs[2];
  int sto_cached[2];

  // cast_set_attention_early_reads: the caller's promise, and whether the last call of this library on the
  // context wrote something the attention reads early (n_tree, masks: cast_select_nodes; kv_len: cast_compact_kv)
  int attn_early;
  int tree_inputs_fresh;
  // work list of the tensor-core attention (one decoded item per CTA), written by a small kernel at the first
  // attention call after the tree or the lengths changed and reused by the calls that follow while the promise
  // above holds and the call's shape is the same (wl_key)
  int32_t* attn_worklist;          // [kAttnWorkListCap][8]
  int wl_valid;
  unsigned long long wl_key[8];

  std::map<int, cast::HostTable>* tables;
  cast::DevTable cur_table;   // table of the current step's batch size (zeros if none)
  int cur_B;
  int next_layer;             // host-side call-order check
};

namespace cast {

#define CAST_CUDA_OK(expr)                      \
  do {                                          \
    cudaError_t _e = (expr);                    \
    if (_e != cudaSuccess) return CAST_ERR_CUDA; \
  } while (0)

inline cast_status launch_status() { return cudaGetLastError() == cudaSuccess ? CAST_OK : CAST_ERR_CUDA; }

// First error wins; later ones are dropped.
__device__ __forceinline__ void report(DevState* st, int code, int detail) {
  if (atomicCAS(&st->status[0], 0, code) == 0) st->status[1] = detail;
}

// Order-preserving map of a float onto unsigned integers (-0 counts as +0).
__device__ __forceinline__ uint32_t ordered_bits(float v) {
  uint32_t b = __float_as_uint(v);
  if (b == 0x80000000u) b = 0u;
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t o) {
  uint32_t b = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
  return __uint_as_float(b);
}
// 64-bit sort key: larger key = (larger logit, then lower token id). Key 0 = "no entry".
__device__ __forceinline__ unsigned long long make_key(float v, int id) {
  return ((unsigned long long)ordered_bits(v) << 32) | (unsigned long long)(0xffffffffu - (uint32_t)id);
}
__device__ __forceinline__ float key_value(unsigned long long k) { return from_ordered_bits((uint32_t)(k >> 32)); }
__device__ __forceinline__ int key_token(unsigned long long k) { return (int)(0xffffffffu - (uint32_t)(k & 0xffffffffu)); }

// select(c) of the cost model read with `min`: grid row in [1, M].
__device__ __forceinline__ int select_grid(int c, int L, int M) {
  int g = c / L;
  if (g > M - 1) g = M - 1;
  return g + 1;
}

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

}  // namespace cast
