// Draft-tree construction: cast_step_begin, cast_tree_expand, cast_select_nodes.
//
// cast_tree_expand is ONE kernel per draft layer, launched as thread-block clusters (the chunks of
// one logits row form a cluster) with programmatic dependent launch between the layers:
//   1. vocabulary sweep - one CTA per chunk: streaming 16-byte loads issued before anything else,
//      online max / sum-exp in base 2, and a list of top-K candidates per warp, filtered against
//      thresholds the CTA's warps share (the K-th largest of the warps' maxima in the first pass, of
//      their best logits afterwards: lower bounds on the CTA's K-th largest, so the result is exact
//      and only a logit or two per warp survives the filter);
//   2. the chunk's top K, maximum and sum go straight into the shared memory of the cluster's
//      first CTA, which merges the row after the cluster barrier (log-sum-exp in fp64, lower-bound
//      merge of the sorted chunk lists) and appends the K children to the node pool;
//   3. the last row-merging CTA of the layer (an atomic ticket; nothing spins) ranks each
//      sequence's candidates, forms the utility u (Eq. 1) and the cost c (Eq. 2), runs Algorithm 1
//      (breadth pruning), the depth-pruning test and the FIFO update, and publishes the retained
//      nodes and the layer's sorted list.
// cast_select_nodes ranks the pool by merging the per-layer sorted lists (binary searches), forms
// the batch-mean utility, runs Algorithm 1 with the target-cost ratio and linearises the tree.
#include <math.h>

#include "cast_internal.h"

using namespace cast;

namespace {

// ------------------------------------------------------------------ expand
struct ExpandParams {
  const void* logits;
  int V, K, W, H, P, layer, nchunks, chunk_elems;
  int prefetch;  // the layer's logits are small enough to be worth asking for ahead of the dependency wait
  double* pool_score;
  int32_t* pool_token;
  int32_t* pool_parent;
  int32_t* pool_depth;
  uint8_t* pool_kept;
  int32_t* retained;
  int32_t* lsort;
  double* lscore;
  DevState* st;
  int32_t* layer_ticket;
  int32_t* seq_ticket;
  double* tail_vs;
  int32_t* tail_sorted;
  int32_t* tail_tok;
  double* fifo_vals;
  int32_t* fifo_cnt;
  int R;
  DevTable tab;
  double C1, C2;
  int enable_bp, enable_dp, ctx_base_mode;
  int32_t* next_tokens;
  int32_t* next_parent_row;
  int32_t* next_count;
  // the step's root tokens and prefix lengths (read by layer 1, which also resets the per-step state)
  const int32_t* root_token;
  const int32_t* kv_len;
};

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
    for (int i = 0; i < 4; ++i) {  // bf16 -> fp32 is a 16-bit shift
      out[2 * i] = __uint_as_float(w[i] << 16);
      out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// log2(e) split into a float just below it and a positive residual: x * log2(e) to better than one ulp
// of the product, and -inf logits stay -inf through both FMAs (no inf - inf)
// Packed fp32 pairs: one instruction, two lanes of the FMA pipe, the same IEEE results per element.
__device__ __forceinline__ unsigned long long pack2(float a, float b) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
constexpr float kLog2eHi = 1.4426950216293335f;
constexpr float kLog2eLo = 1.925963033500011e-08f;  // log2(e) - kLog2eHi

// exp(s) for s <= 0 to about 1.2e-7 relative: the product with log2(e) and the integer part in fp64, the
// fractional power by the fp32 unit, exact scaling. (A node value needs no more: the decision margins that
// the parity contract asks for are 2e-6 relative.)
__device__ __forceinline__ double fast_exp_neg(double s) {
  const double t = s * 1.4426950408889634074;
  if (!(t > -1000.0)) return 0.0;
  const double n = floor(t);
  return ldexp((double)ex2f((float)(t - n)), (int)n);
}
// log2(S), S > 0, to about 1e-7 absolute: exact exponent split, fp32 logarithm of the mantissa
__device__ __forceinline__ double fast_log2(double S) {
  int e;
  const double m = frexp(S, &e);
  return (double)e + (double)log2f((float)m);
}

// ---- thread-block cluster primitives (a logits row is swept by one cluster)
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_u64(uint32_t addr, unsigned long long v) {
  asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void st_cluster_f64(uint32_t addr, double v) {
  asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(addr), "d"(v) : "memory");
}
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// Programmatic dependent launch (both are no-ops for a grid launched without the attribute).
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// State fields the layer tail needs; every CTA reads them at its start (same cache lines as the row
// count it needs anyway), so the tail itself starts without a round trip to memory.
struct TailState {
  int ctx_sum, n0, kept_total;
  double u_last;
};

// The ticket of the "last CTA" pattern: the caller has passed a CTA barrier after its global
// writes; one thread takes the ticket with release-acquire semantics (cumulative over the CTA's writes).
__device__ __forceinline__ bool take_ticket(int32_t* counter, int expected, int* flag_s) {
  if (threadIdx.x == 0) {
    // one acquire-release atomic at device scope: releases this CTA's writes (the barrier before the
    // call made them this thread's to release), acquires those of the CTAs that came earlier
    int t;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(t) : "l"(counter) : "memory");
    const int last = (t == expected - 1);
    if (last) *counter = 0;
    *flag_s = last;
  }
  __syncthreads();
  return *flag_s != 0;
}

// Layer tail (Eq. 1, Eq. 2, Algorithm 1, depth pruning) in two parts. tail_rank orders the candidates of
// some sequences and is what costs time with many sequences; tail_decide is the batch-wide rest. With up to
// four sequences the last CTA of the layer runs both from shared memory; with more, the last CTA of every
// sequence ranks that sequence (so the sequences are ranked in parallel) and leaves the first n sorted
// nodes in global memory, and the last of those CTAs decides.

// Up to this many sequences the one-CTA tail is faster than a second ticket.
constexpr int kTailSingleMaxB = 4;

// a / b for 0 <= a < 2^20 and 1 <= b <= 2^10 through the fp32 reciprocal (inv_b = 1.f / b) with one correction step:
// the integer division by a run-time divisor is some twenty instructions, and the ranking below does several per
// thread in a phase whose time is what its instructions take to issue.
__device__ __forceinline__ int div_small(int a, int b, float inv_b) {
  int q = (int)((float)a * inv_b);
  const int r = a - q * b;
  q += (r >= b) ? 1 : 0;
  q -= (r < 0) ? 1 : 0;
  return q;
}

// Candidates Algorithm 1 looks at: the first n of the sorted list.
__device__ __forceinline__ int tail_width(const ExpandParams& p, int n_prev) {
  const int Ni = n_prev * p.K;
  int n = Ni < p.W ? Ni : p.W;
  if ((p.enable_bp || p.enable_dp) && p.tab.Ntab < n) n = p.tab.Ntab;
  return n;
}

// Ranks the layer's candidates of the sequences [b_begin, b_begin + b_count): writes every sequence's sorted
// list for the rerank (lsort, lscore) and, for rank < n, pool index, token and value to sorted_o, stok_o,
// vs_o at [b * CAST_MAX_WIDTH + rank] (shared or global memory).
__device__ __forceinline__ void tail_rank(const ExpandParams& p, int b_begin, int b_count, int n, int n_prev, int base,
                                          unsigned char* scratch, int* sorted_o, int* stok_o, double* vs_o) {
  const int tid = threadIdx.x, nt = blockDim.x;
  const int K = p.K, P = p.P;
  const int Ni = n_prev * K;
  double* sc = reinterpret_cast<double*>(scratch);              // 1024 scores
  int* tk = reinterpret_cast<int*>(scratch + 8192);             // 1024 tokens
  int* rank_s = reinterpret_cast<int*>(scratch + 12288);        // 1024 ranks
  const int group = 1024 / Ni;                                  // sequences ranked per pass
  const float inv_Ni = 1.f / (float)Ni, inv_K = 1.f / (float)K;
#pragma unroll 1
  for (int b0 = 0; b0 < b_count; b0 += group) {
    const int nb = (b_count - b0) < group ? (b_count - b0) : group;
    const int tot = nb * Ni;
    for (int i = tid; i < tot; i += nt) {
      const int bl = div_small(i, Ni, inv_Ni), ci = i - bl * Ni;
      const size_t o = (size_t)(b_begin + b0 + bl) * P + base + ci;
      sc[i] = __ldcg(p.pool_score + o);
      tk[i] = __ldcg(p.pool_token + o);
      rank_s[i] = 0;
    }
    __syncthreads();
    // Rank under the order (value desc, token asc, creation order). Every logits row contributed its K
    // children already in that order, so the rank of a candidate is, summed over the rows of its sequence,
    // the number of that row's children that come first: one lower-bound search per (candidate, row) pair (in
    // its own row it finds its own position). The pairs are spread densely over the threads - what this phase
    // costs is the warp instructions it issues, so no lane works on a row or a step that does not exist - two
    // per thread in step so that their shared-memory loads overlap; the counts meet in shared memory.
    const int pairs = tot * n_prev;
    const float inv_tot = 1.f / (float)tot;
    int h0 = 1;
    while (2 * h0 - 1 < K) h0 <<= 1;  // the search's first stride: positions up to 2 h0 - 1 >= K are reachable
#pragma unroll 1
    for (int it0 = tid; it0 < pairs; it0 += 2 * nt) {
      int ii[2], rs[2], rowb[2], r1[2], t2[2], pos[2] = {0, 0};
      double s2[2];
      bool act[2];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int it = it0 + q * nt;
        act[q] = it < pairs;
        const int itc = act[q] ? it : 0;
        // (row-major: the lanes of a warp search one row for consecutive candidates, so their shared-memory loads
        // fall on that row's K entries and their counts go to different words)
        rs[q] = div_small(itc, tot, inv_tot);    // the row searched
        ii[q] = itc - rs[q] * tot;               // the candidate (index over the sequences of this pass)
        const int ci = ii[q] - div_small(ii[q], Ni, inv_Ni) * Ni;
        r1[q] = div_small(ci, K, inv_K);         // the candidate's own row
        rowb[q] = ii[q] - ci + rs[q] * K;  // first child of the searched row, same sequence
        s2[q] = sc[ii[q]];
        t2[q] = tk[ii[q]];
      }
#pragma unroll 1
      for (int half = h0; half >= 1; half >>= 1) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int idx = pos[q] + half - 1;
          const bool valid = idx < K;
          const int at = rowb[q] + (valid ? idx : 0);
          const double sj = sc[at];
          const int tj = tk[at];
          const bool first = valid && ((sj > s2[q]) || (sj == s2[q] && (tj < t2[q] || (tj == t2[q] && rs[q] < r1[q]))));
          pos[q] += first ? half : 0;
        }
      }
#pragma unroll
      for (int q = 0; q < 2; ++q)
        if (act[q] && pos[q] != 0) atomicAdd(&rank_s[ii[q]], pos[q]);
    }
    __syncthreads();
#pragma unroll 1
    for (int i = tid; i < tot; i += nt) {
      const int bl = div_small(i, Ni, inv_Ni), ci = i - bl * Ni, rank = rank_s[i];
      const int bg = b_begin + b0 + bl;
      const double s = sc[i];
      const size_t o = (size_t)bg * P + base + rank;
      p.lsort[o] = base + ci;  // the layer's sorted list, for the rerank
      p.lscore[o] = s;
      if (rank < n) {
        sorted_o[bg * CAST_MAX_WIDTH + rank] = base + ci;
        stok_o[bg * CAST_MAX_WIDTH + rank] = tk[i];
        vs_o[bg * CAST_MAX_WIDTH + rank] = fast_exp_neg(s);
      }
    }
    __syncthreads();
  }
}

// The batch-wide part: Eq. 1 over the sequences' first n sorted values, Eq. 2, Algorithm 1, the depth test,
// the state for the next layer and the layer's outputs. GLOBAL: the inputs were written to global memory by
// other CTAs (read past L1).
template <bool GLOBAL>
__device__ __forceinline__ void tail_decide(const ExpandParams& p, const TailState& ts, int B, int n, int n_prev, int base,
                                            const int* sorted_i, const int* stok_i, const double* vs_i) {
  __shared__ double vbar[CAST_MAX_WIDTH], u[CAST_MAX_WIDTH], c[CAST_MAX_WIDTH];
  __shared__ int s_ni, s_next, s_n0;
  const int tid = threadIdx.x, nt = blockDim.x;
  DevState* st = p.st;
  const int K = p.K, W = p.W, P = p.P;
  const int Ni = n_prev * K;
  const bool need_cost = p.enable_bp || p.enable_dp;
  const double u_last = ts.u_last;
  int n0 = ts.n0;
  if (p.layer == 1) {
    // The first layer of a step also starts the step (cast_step_begin launches nothing): the padded context
    // length n_0 = max_b kv_len[b] and every sequence's root node (value 1, depth 0) at pool index 0.
    static_assert(CAST_MAX_BATCH <= 64, "two sequences per lane");
    if (tid < 32) {
      int m = max(tid < B ? p.kv_len[tid] : 0, tid + 32 < B ? p.kv_len[tid + 32] : 0);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
      if (tid == 0) s_n0 = m;
    }
    for (int b = tid; b < B; b += nt) {
      const size_t o = (size_t)b * P;
      p.pool_score[o] = 0.0;
      p.pool_token[o] = p.root_token[b];
      p.pool_parent[o] = -1;
      p.pool_depth[o] = 0;
      p.pool_kept[o] = 1;
      p.lsort[o] = 0;
      p.lscore[o] = 0.0;
    }
    __syncthreads();
    n0 = s_n0;
  }
  // Eq. 1: batch mean of the rank-wise values, then prefix sums; Eq. 2 needs one table row
  if (tid < n) {
    double c_mine = 0.0;
    if (need_cost) {
      const int ctx = ts.ctx_sum + (p.ctx_base_mode ? n0 : 0);
      const int g = select_grid(ctx, p.tab.L, p.tab.M);
      c_mine = p.tab.fD[(size_t)(g - 1) * p.tab.Ntab + tid] / p.tab.fT[(size_t)(g - 1) * p.tab.Ntab];
    }
    if (!GLOBAL) {
      double a = 0.0;
#pragma unroll 1
      for (int b = 0; b < B; ++b) a += vs_i[b * CAST_MAX_WIDTH + tid];
      vbar[tid] = a / (double)B;
    }
    c[tid] = c_mine;
  }
  if (GLOBAL) {
    // many sequences: warp j sums rank j over the sequences, two per lane, then a fixed shuffle tree
    static_assert(kSweepThreads / 32 >= CAST_MAX_WIDTH && CAST_MAX_BATCH <= 64, "one warp per rank, two sequences per lane");
    const int j = tid >> 5, lane = tid & 31;
    if (j < n) {
      double a = (lane < B ? __ldcg(vs_i + lane * CAST_MAX_WIDTH + j) : 0.0) +
                 (lane + 32 < B ? __ldcg(vs_i + (lane + 32) * CAST_MAX_WIDTH + j) : 0.0);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
      if (lane == 0) vbar[j] = a / (double)B;
    }
  }
  __syncthreads();
  if (tid < 32) {  // inclusive scan of at most 16 values
    double a = tid < n ? vbar[tid] : 0.0;
#pragma unroll
    for (int d = 1; d < CAST_MAX_WIDTH; d <<= 1) {
      const double t = __shfl_up_sync(0xffffffffu, a, d);
      if (tid >= d) a += t;
    }
    if (tid < n) u[tid] = a;
  }
  __syncthreads();
  // Algorithm 1: mark[j] survives iff no earlier i has (u_j - u_i) < C1 (c_j - c_i); n_i = the largest
  // marked index. n <= CAST_MAX_WIDTH <= 32: one warp, the marks as a ballot.
  if (tid < 32) {
    int ok = tid < n ? 1 : 0;
    if (p.enable_bp && tid < n) {
      const double uj = u[tid], cj = c[tid];
#pragma unroll 4
      for (int i = 0; i < tid; ++i)
        ok &= !((uj - u[i]) < p.C1 * (cj - c[i]));
    }
    const unsigned marks = __ballot_sync(0xffffffffu, ok != 0);
    if (tid == 0) s_ni = marks != 0u ? 32 - __clz(marks) : 1;
  }
  __syncthreads();
  if (tid == 0) {
    const int n_i = s_ni;
    bool go = true;
    if (p.enable_dp) {
      if (p.layer >= 2) {  // gain ratio of the previous layer goes into its buffer, FIFO
        const double phi = u[n_i - 1] / u_last;
        double* A = p.fifo_vals + (size_t)(p.layer - 2) * p.R;
        int cnt = p.fifo_cnt[p.layer - 2];
        if (cnt < p.R) {
          A[cnt++] = phi;
        } else {
          for (int k = 1; k < p.R; ++k) A[k - 1] = A[k];
          A[p.R - 1] = phi;
        }
        p.fifo_cnt[p.layer - 2] = cnt;
      }
      if (p.layer < p.H) {  // generate layer i+1 only if Avg(A_i) * u / c >= C2
        const double* A = p.fifo_vals + (size_t)(p.layer - 1) * p.R;
        const int cnt = p.fifo_cnt[p.layer - 1];
        double a = 0.0;
        for (int k = 0; k < cnt; ++k) a += A[k];
        const double alpha = a / (double)cnt;
        go = (alpha * u[n_i - 1] / c[n_i - 1]) >= p.C2;
      }
    }
    s_next = (p.layer < p.H && go) ? n_i : 0;
    if (p.layer == 1) {  // per-step state (rows[]: a later layer that is never reached must read 0)
      st->B = B;
      st->n0 = n0;
      st->n_tree = 0;
      st->n_hist[0] = 1;
      st->layer_base[0] = 0;
      st->layer_n[0] = 1;
      for (int i = 2; i <= CAST_MAX_DEPTH; ++i) {
        st->n_hist[i] = 0;
        st->layer_base[i] = 0;
        st->layer_n[i] = 0;
      }
      for (int i = 0; i < CAST_MAX_DEPTH + 2; ++i) st->rows[i] = (i == 1) ? 1 : 0;
    }
    st->rows[p.layer + 1] = s_next;
    st->n_hist[p.layer] = n_i;
    st->layer_base[p.layer] = base;
    st->layer_n[p.layer] = Ni;
    st->ctx_sum = ts.ctx_sum + n_i;
    st->kept_total = ts.kept_total + n_i;
    st->u_last = u[n_i - 1];
    st->pool_size = base + Ni;
    st->layers_done = p.layer;
    *p.next_count = s_next;
  }
  __syncthreads();
  const int n_i = s_ni;
#pragma unroll 1
  for (int i = tid; i < B * W; i += nt) {
    const int b = i / W, s = i % W;
    int tok = -1, prow = -1;
    if (s < n_i) {
      const int idx = GLOBAL ? __ldcg(sorted_i + b * CAST_MAX_WIDTH + s) : sorted_i[b * CAST_MAX_WIDTH + s];
      tok = GLOBAL ? __ldcg(stok_i + b * CAST_MAX_WIDTH + s) : stok_i[b * CAST_MAX_WIDTH + s];
      prow = (idx - base) / K;
      p.retained[b * W + s] = idx;
      p.pool_kept[(size_t)b * P + idx] = 1;
    }
    p.next_tokens[i] = tok;
    p.next_parent_row[i] = prow;
  }
}

// MINB = 2 compiles the same code for two CTAs per SM (half the registers): for launches with more CTAs than
// SMs, where a second resident CTA hides the first one's latencies; MINB = 1 is for the short launches.
template <typename T, int MINB>
__global__ void __launch_bounds__(kSweepThreads, MINB) expand_kernel(const ExpandParams p) {
  __shared__ __align__(16) unsigned char scratch[kCandCap * 8];  // the warps' key lists and the short list; later the tail's arrays
  __shared__ unsigned long long topk[CAST_MAX_TOP_K];
  __shared__ float red_f[kSweepThreads / 32];
  __shared__ double red_d[kSweepThreads / 32];
  __shared__ int sorted[kTailSingleMaxB * CAST_MAX_WIDTH];  // small batches: pool indices of the first sorted candidates
  __shared__ int s_flag, short_n;
  __shared__ float pass_heads[2][kSweepThreads / 32];  // the warps' largest logits after a pass (see cta_bound)
  __shared__ float pass_wmax[kSweepThreads / 32];                   // the warps' maxima of the first pass
  static_assert(CAST_MAX_TOP_K <= kSweepThreads / 32, "the K-th largest of the warps' maxima needs K <= warps");
  // filled in the first CTA of the row's cluster by all CTAs of the cluster: chunk c's top-K keys
  // (descending), maximum (log2 units) and sum of 2^(. - maximum)
  __shared__ unsigned long long row_keys[kSweepMaxChunks * CAST_MAX_TOP_K];
  __shared__ float row_max[kSweepMaxChunks];
  __shared__ double row_sum[kSweepMaxChunks];
  unsigned long long* cand = reinterpret_cast<unsigned long long*>(scratch);

  const int chunk = blockIdx.x, r = blockIdx.y, b = blockIdx.z, B = gridDim.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  DevState* st = p.st;
  const int K = p.K;
  const int row = b * p.W + r;
  const T* x = reinterpret_cast<const T*>(p.logits) + (size_t)row * p.V;
  const int begin = chunk * p.chunk_elems;
  const int end = min(begin + p.chunk_elems, p.V);
  constexpr int VEC = Vec<T>::N;
  constexpr int NV = kSweepEpt / VEC;
  const bool aligned = (reinterpret_cast<uintptr_t>(x) & 15) == 0;  // chunk starts are multiples of 8 logits

  // the first pass of logits is requested before the state is read (every row r < W exists in memory):
  // one memory round trip for both
  float xv[kSweepEpt];
  auto load_pass = [&](int sub) {
    if (aligned && sub + kSweepSub <= end) {  // a full pass: no per-vector checks
#pragma unroll
      for (int v = 0; v < NV; ++v) Vec<T>::load(x + sub + (v * kSweepThreads + tid) * VEC, xv + v * VEC);
      return;
    }
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const int idx = sub + (v * kSweepThreads + tid) * VEC;
      if (aligned && idx + VEC <= end) {
        Vec<T>::load(x + idx, xv + v * VEC);
      } else {
#pragma unroll
        for (int e = 0; e < VEC; ++e) xv[v * VEC + e] = (idx + e < end) ? to_float(x[idx + e]) : -INFINITY;
      }
    }
  };
  // Programmatic dependent launch: this grid may have become resident while the previous kernel of the
  // stream was still finishing. Nothing that kernel may have written is read above this line - not the
  // logits either: in a serving loop the previous kernel is the draft model's, and it writes them. What a
  // CTA may do is ask the L2 cache for its chunk: a prefetch returns no value, and a line that the previous
  // kernel writes afterwards is written in that same cache, so the loads below see it. When the previous kernel
  // is not the one that writes the logits (layers queued back to back) the first pass then costs a round trip
  // to L2 instead of one to HBM; rows that turn out not to exist are fetched for nothing, hence only for small
  // layers.
  if (p.prefetch) {
    const char* cb = reinterpret_cast<const char*>(x + begin);
    const int bytes = (end - begin) * (int)sizeof(T);
#pragma unroll 1
    for (int off = tid * 128; off < bytes; off += kSweepThreads * 128)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(cb + off));
  }
  grid_dependency_wait();
  grid_launch_dependents();  // the next grid may now take the SMs this one leaves idle
  load_pass(begin);
  // what the layer tail needs of the state is read now, together with the row count: one round trip.
  // (Layer 1 starts the step: one row per sequence, the root at pool index 0 with value 1.)
  int n_prev = 1, base = 1;
  TailState ts;
  ts.ctx_sum = 0;
  ts.n0 = 0;  // layer 1: the deciding CTA works it out from kv_len
  ts.kept_total = 1;
  ts.u_last = 1.0;
  if (p.layer > 1) {
    n_prev = st->rows[p.layer];
    ts.ctx_sum = st->ctx_sum;
    ts.n0 = st->n0;
    ts.kept_total = st->kept_total;
    ts.u_last = st->u_last;
    base = st->pool_size;
  }
  if (n_prev == 0) {
    if (chunk == 0 && r == 0 && b == 0 && tid == 0) *p.next_count = 0;
    return;
  }
  if (r >= n_prev) return;
  // the parent of this row's children and its log-value (only the row's last CTA uses them: fetched now,
  // off the critical path)
  int parent = 0;
  double parent_score = 0.0;
  if (p.layer > 1) {
    parent = p.retained[b * p.W + r];
    parent_score = p.pool_score[(size_t)b * p.P + parent];
  }

  float M2 = -INFINITY, s_run = 0.f;  // running maximum (log2 units) and sum of 2^(x log2e - M2)
  // Every warp keeps the exact top K of the logits it has seen, as a descending list in shared memory;
  // the warps never meet during the sweep. `have` (warp-uniform) is the list's length, thr_key its K-th
  // key (0 while it is shorter than K).
  constexpr int kWarpCap = 64;
  constexpr int kWarps = kSweepThreads / 32;
  unsigned long long* wlist = cand + warp * kWarpCap;
  int have = 0;
  unsigned long long thr_key = 0ull;
  // A lower bound on the CTA's K-th largest logit that all warps share from the second pass on: the K-th
  // largest of the warps' best logits so far (K of the CTA's logits are at least that large). A warp's own K-th
  // key only knows the warp's sixteenth of the data; against this bound few logits of a later pass reach any
  // list at all, so the exact tests, the appends and the re-ranking below mostly do not run. (A logit of the
  // CTA's final top K is >= every such bound, and a warp drops it only for K better ones: the chunk result is
  // exact. The bound is a value, not a key: logits equal to it pass, which only lengthens a list.)
  float cta_bound = -INFINITY;
  int pass = 0;
  const int npass = (end - begin + kSweepSub - 1) / kSweepSub;

  for (int sub = begin; sub < end; sub += kSweepSub, ++pass) {
    if (sub != begin) load_pass(sub);
    // The bound is refreshed where it still moves: before the second pass (from the first pass's threshold to the
    // K-th largest of sixteen warps' best it rises a great deal) and, in long chunks, before the third. Later it
    // hardly rises, the warps' own K-th keys have caught up, and the refresh - a CTA barrier and a rank of 16 heads
    // in every warp, about a third of a pass's instructions - costs more than the few extractions it saves
    // (batch 64, eight passes: 302 -> 278 us per tree build; batch 16, four passes: 171 -> 166).
    if (pass == 1 || (pass == 2 && npass >= 6)) {
      float* hd = pass_heads[pass & 1];
      if (lane == 0) hd[warp] = have > 0 ? key_value(wlist[0]) : -INFINITY;
      __syncthreads();
      const float head = lane < kWarps ? hd[lane] : -INFINITY;
      int rh = 0;
#pragma unroll
      for (int j = 0; j < kWarps; ++j) {
        const float o = __shfl_sync(0xffffffffu, head, j);
        rh += (o > head) || (o == head && j < lane);  // equal heads in lane order: ranks 0..15 are distinct
      }
      const unsigned who = __ballot_sync(0xffffffffu, lane < kWarps && rh == K - 1);
      const float bnd = __shfl_sync(0xffffffffu, head, who != 0u ? __ffs(who) - 1 : 0);
      cta_bound = fmaxf(cta_bound, bnd);
    }
    // (the maxima of the four groups of eight slots on the way: the extraction below looks only into the groups
    // that hold a passer)
    float gmax[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      gmax[g] = xv[8 * g];
#pragma unroll
      for (int j = 1; j < 8; ++j) gmax[g] = fmaxf(gmax[g], xv[8 * g + j]);
    }
    const float tmax = fmaxf(fmaxf(gmax[0], gmax[1]), fmaxf(gmax[2], gmax[3]));
    const float t2 = tmax * kLog2eHi;
    if (t2 > M2) {
      s_run *= ex2f(M2 - t2);
      M2 = t2;
    }
    if (M2 > -INFINITY) {
      // x * log2(e) - M2 with log2(e) in two parts (the product is exact to fp32's last bit and beyond), two
      // logits per instruction; NaN and +inf logits poison the sum
      const unsigned long long hi2 = pack2(kLog2eHi, kLog2eHi), lo2 = pack2(kLog2eLo, kLog2eLo), nm2 = pack2(-M2, -M2);
      unsigned long long acc2 = pack2(0.f, 0.f);
#pragma unroll
      for (int i = 0; i < kSweepEpt; i += 2) {
        const unsigned long long x2 = pack2(xv[i], xv[i + 1]);
        float e0, e1;
        unpack2(fma2(x2, hi2, fma2(x2, lo2, nm2)), e0, e1);
        acc2 = add2(acc2, pack2(ex2f(e0), ex2f(e1)));
      }
      float a0, a1;
      unpack2(acc2, a0, a1);
      s_run += a0 + a1;
    }
    // filter threshold: the warp's exact K-th key once it has K, else the K-th largest of the lanes'
    // maxima of this pass (at least K of the warp's logits are >= it)
    float thr_val;
    const unsigned long long gate = thr_key;  // keys at or below the warp's own K-th cannot matter
    if (pass == 0) {
      // nothing is known yet: the K-th largest of the 16 warps' maxima (K <= 16 of the CTA's logits are at
      // least that large). Against it one or two logits per warp pass; against the K-th largest of a warp's
      // own lane maxima, which needs no barrier but a 15-stage sorting network, K to 2K per warp did.
      float wm = tmax;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
      float* wmax = pass_wmax;
      if (lane == 0) wmax[warp] = wm;
      __syncthreads();
      const float mine = lane < kWarps ? wmax[lane] : -INFINITY;
      int rh = 0;
#pragma unroll
      for (int j = 0; j < kWarps; ++j) {
        const float o = __shfl_sync(0xffffffffu, mine, j);
        rh += (o > mine) || (o == mine && j < lane);  // equal maxima in lane order: ranks 0..15 are distinct
      }
      const unsigned who = __ballot_sync(0xffffffffu, lane < kWarps && rh == K - 1);
      thr_val = __shfl_sync(0xffffffffu, mine, who != 0u ? __ffs(who) - 1 : 0);
    } else if (gate == 0ull && !(cta_bound > -INFINITY)) {
      float kx = tmax;
#pragma unroll
      for (int k = 2; k <= 32; k <<= 1)
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
          const float o = __shfl_xor_sync(0xffffffffu, kx, j);
          const bool desc = ((lane & k) == 0), low = ((lane & j) == 0);
          kx = (desc == low) ? fmaxf(kx, o) : fminf(kx, o);
        }
      thr_val = __shfl_sync(0xffffffffu, kx, K - 1);
    } else {
      thr_val = gate != 0ull ? fmaxf(key_value(gate), cta_bound) : cta_bound;
    }
    // Few logits pass, and against the shared thresholds most passes of a warp have none: one vote on the
    // lanes' maxima settles that. Otherwise the same vote per group of eight slots, and in a group with a passer
    // every lane marks its passing slots in a bit mask, the warp takes the union with one reduction and walks its
    // set bits (a loop over the set bits only: unrolled over all slots, the tests and reconvergence points of the
    // empty ones were most of the sweep's time); a slot's logit is picked out of the group's registers by three
    // rounds of warp-uniform selects, takes the exact test on the full key and is appended to the warp's list.
    // (The order of the appends does not matter: the list is ranked afterwards.)
    const int have0 = have;
    if (__any_sync(0xffffffffu, tmax >= thr_val)) {
      static_assert(kSweepEpt == 32, "four groups of eight slots");
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        if (!__any_sync(0xffffffffu, gmax[g] >= thr_val)) continue;
        unsigned mine_mask = 0u;
#pragma unroll
        for (int j = 0; j < 8; ++j) mine_mask |= (xv[8 * g + j] >= thr_val) ? (1u << j) : 0u;
        unsigned any_mask = __reduce_or_sync(0xffffffffu, mine_mask);
#pragma unroll 1
        while (any_mask != 0u) {
          const int j = __ffs(any_mask) - 1;
          any_mask &= any_mask - 1u;
          const bool b0 = (j & 1) != 0, b1 = (j & 2) != 0, b2 = (j & 4) != 0;
          float s4[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) s4[q] = b0 ? xv[8 * g + 2 * q + 1] : xv[8 * g + 2 * q];
          const float s2a = b1 ? s4[1] : s4[0], s2b = b1 ? s4[3] : s4[2];
          const float xi = b2 ? s2b : s2a;
          const int i = 8 * g + j;
          const int id = sub + ((i / VEC) * kSweepThreads + tid) * VEC + (i % VEC);
          const unsigned long long key = make_key(xi, id);
          const bool ok = xi >= thr_val && id < end && key > gate;
          const unsigned m = __ballot_sync(0xffffffffu, ok);
          const int pos = have + __popc(m & ((1u << lane) - 1u));
          if (ok && pos < kWarpCap) wlist[pos] = key;
          have += __popc(m);
        }
      }
    }
    __syncwarp();
    if (have > kWarpCap) {
      // flood (a mass of ties at the threshold): K rounds of "largest key below the last one taken" over
      // the old list and this pass's logits; lane r keeps the r-th result
      unsigned long long bound = ~0ull, mine = 0ull;
      int n = 0;
#pragma unroll 1
      for (int round = 0; round < K; ++round) {
        unsigned long long best = 0ull;
#pragma unroll
        for (int i = 0; i < kSweepEpt; ++i) {
          const int id = sub + ((i / VEC) * kSweepThreads + tid) * VEC + (i % VEC);
          if (id < end && xv[i] == xv[i]) {
            const unsigned long long k2 = make_key(xv[i], id);
            if (k2 < bound && k2 > best) best = k2;
          }
        }
        if (lane < have0) {
          const unsigned long long k2 = wlist[lane];
          if (k2 < bound && k2 > best) best = k2;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
          best = other > best ? other : best;
        }
        if (best == 0ull) break;
        if (lane == round) mine = best;
        ++n;
        bound = best;
      }
      __syncwarp();
      if (lane < n) wlist[lane] = mine;
      have = n;
      __syncwarp();
    } else if (have == have0 + 1) {
      // one newcomer (the usual case): the old entries are in order, so it is an insertion - the newcomer's rank is
      // the number of larger keys (one vote), the smaller ones move down one place, the K-th of K falls off
      const unsigned long long nk = wlist[have0];
      const unsigned long long mine = lane < have0 ? wlist[lane] : 0ull;
      const int rnk = __popc(__ballot_sync(0xffffffffu, lane < have0 && mine > nk));
      __syncwarp();
      if (lane < have0 && lane >= rnk && lane + 1 < K) wlist[lane + 1] = mine;
      if (lane == 0 && rnk < K) wlist[rnk] = nk;
      have = have < K ? have : K;
      __syncwarp();
    } else if (have > have0) {
      // exact order of the list (old entries and newcomers, at most 64): rank by counting, keys are distinct
      const int n = have;
      const unsigned long long k0 = lane < n ? wlist[lane] : 0ull;
      const unsigned long long k1 = lane + 32 < n ? wlist[lane + 32] : 0ull;
      int r0 = 0, r1 = 0;
#pragma unroll 4
      for (int j = 0; j < n; ++j) {
        const unsigned long long kj = wlist[j];
        r0 += (kj > k0);
        r1 += (kj > k1);
      }
      __syncwarp();
      if (lane < n && r0 < K) wlist[r0] = k0;
      if (lane + 32 < n && r1 < K) wlist[r1] = k1;
      have = n < K ? n : K;
      __syncwarp();
    }
    thr_key = have == K ? wlist[K - 1] : 0ull;
  }

  // chunk result: the top K of the warps' lists (each in descending order; the rank of a key is the
  // number of larger keys, list by list: a lower-bound search each, two lanes per key slot), the
  // maximum and the sum of 2^(. - maximum) in fp64. It goes straight into the shared memory of the
  // cluster's first CTA, which merges the row.
  {
    if (lane >= have && lane < CAST_MAX_TOP_K) wlist[lane] = 0ull;  // short lists end in "no entry"
    float Mw = M2;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Mw = fmaxf(Mw, __shfl_xor_sync(0xffffffffu, Mw, o));
    double sd = (M2 > -INFINITY) ? (double)s_run * (double)ex2f(M2 - Mw) : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sd += __shfl_xor_sync(0xffffffffu, sd, o);
    if (lane == 0) {
      red_f[warp] = Mw;
      red_d[warp] = sd;
    }
    if (tid < K) topk[tid] = 0ull;
    if (tid == 0) short_n = 0;  // length of the CTA's short list
    __syncthreads();
    // The K-th largest of the warps' list heads bounds the CTA's top K from below (every list is in
    // descending order), so only keys at or above it can belong: a dozen or so. Every warp finds that
    // bound by itself (16 heads, one per lane), appends its survivors to a short list with one atomic,
    // and the first warp ranks the short list by counting.
    unsigned long long bound;
    {
      const unsigned long long head = lane < kWarps ? cand[lane * kWarpCap] : 0ull;
      int rh = 0;
#pragma unroll
      for (int j = 0; j < kWarps; ++j) rh += (__shfl_sync(0xffffffffu, head, j) > head);
      bound = (rh == K - 1) ? head : 0ull;  // heads are distinct unless 0 ("no entry")
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, bound, o);
        bound = other > bound ? other : bound;
      }
    }
    unsigned long long* shortlist = cand + kWarps * kWarpCap;  // at most kWarps * K keys
    {
      const unsigned long long key = lane < have ? wlist[lane] : 0ull;
      const bool keep = key != 0ull && key >= bound;
      const unsigned m = __ballot_sync(0xffffffffu, keep);
      int basepos = 0;
      if (lane == 0 && m != 0u) basepos = atomicAdd(&short_n, __popc(m));
      basepos = __shfl_sync(0xffffffffu, basepos, 0);
      if (keep) shortlist[basepos + __popc(m & ((1u << lane) - 1u))] = key;
    }
    __syncthreads();
    if (warp == 0) {
      const int n = short_n;  // <= kWarps * K = 256: up to 8 keys per lane
#pragma unroll 1
      for (int i0 = 0; i0 < n; i0 += 32) {
        const int i = i0 + lane;
        const unsigned long long key = i < n ? shortlist[i] : ~0ull;
        int rk2 = 0;
#pragma unroll 4
        for (int j = 0; j < n; ++j) rk2 += (shortlist[j] > key);
        if (i < n && rk2 < K) topk[rk2] = key;
      }
    }
    // meanwhile the last warp folds the warps' (maximum, sum) pairs
    float M = -INFINITY;
    double S = 0.0;
    if (warp == kWarps - 1) {
      const float Ml = lane < kWarps ? red_f[lane] : -INFINITY;
      const double Sl = lane < kWarps ? red_d[lane] : 0.0;
      M = Ml;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
      S = Ml > -INFINITY ? Sl * (double)ex2f(Ml - M) : 0.0;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) S += __shfl_xor_sync(0xffffffffu, S, o);
    }
    __syncthreads();
    if (p.nchunks == 1) {
      if (tid < K) row_keys[tid] = topk[tid];
      if (tid == kSweepThreads - 32) {
        row_max[0] = M;
        row_sum[0] = S;
      }
    } else {
      if (tid < K) st_cluster_u64(map_to_rank(smem_addr(&row_keys[chunk * CAST_MAX_TOP_K + tid]), 0u), topk[tid]);
      if (tid == kSweepThreads - 32) {
        st_cluster_f32(map_to_rank(smem_addr(&row_max[chunk]), 0u), M);
        st_cluster_f64(map_to_rank(smem_addr(&row_sum[chunk]), 0u), S);
      }
    }
  }

  // ---- row merge by the first CTA of the row's cluster
  if (p.nchunks > 1) {
    cluster_arrive_release();
    if (chunk != 0) return;  // the results are on their way; the first CTA waits for them
    cluster_wait_acquire();
  } else {
    __syncthreads();
  }
  // the row's top K out of the chunks' lists (each in descending order): the rank of a key is its
  // position in its own list plus, for every other list, the number of larger keys there (a binary
  // search each; in its own list it finds its own position). Neighbouring lanes share a key slot.
  if (p.nchunks > 1) {  // (a row of one chunk has its top K in `topk` already)
  if (tid < K) topk[tid] = 0ull;
  __syncthreads();
  {
    constexpr int kLps = kSweepThreads / (kSweepMaxChunks * CAST_MAX_TOP_K);  // lanes per key slot: one pass
    constexpr int kLpl = kSweepMaxChunks / kLps;                              // lists per lane
    static_assert(kLps >= 1 && kLps <= 8 && kLps * kLpl == kSweepMaxChunks, "lanes of a slot cover the lists");
    const int slot = tid / kLps, sub = tid % kLps;
    const int c1 = slot >> 4, t = slot & 15;  // slot = list * CAST_MAX_TOP_K + position
    const bool act = c1 < p.nchunks && t < K;
    const unsigned long long key = act ? row_keys[slot] : 0ull;
    int pos[kLpl];
#pragma unroll
    for (int q = 0; q < kLpl; ++q) pos[q] = 0;
#pragma unroll
    for (int half = 16; half >= 1; half >>= 1) {
#pragma unroll
      for (int q = 0; q < kLpl; ++q) {
        const int c2 = sub + kLps * q;
        const int idx = pos[q] + half - 1;
        const bool valid = act && c2 < p.nchunks && idx < K;
        const unsigned long long other = row_keys[valid ? c2 * CAST_MAX_TOP_K + idx : 0];
        pos[q] += (valid && other > key) ? half : 0;
      }
    }
    int cnt = 0;
#pragma unroll
    for (int q = 0; q < kLpl; ++q) cnt += pos[q];
#pragma unroll
    for (int o = kLps >> 1; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (act && sub == 0 && cnt < K) topk[cnt] = key;
  }
  __syncthreads();
  }
  if (warp == 0) {
    float M0 = -INFINITY, M1 = -INFINITY;
    double S0 = 0.0, S1 = 0.0;
    if (lane < p.nchunks) {
      M0 = row_max[lane];
      S0 = row_sum[lane];
    }
    // (d) log-sum-exp over the chunk partials: weights by the fp32 unit, sums in fp64
    float Mr = fmaxf(M0, M1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Mr = fmaxf(Mr, __shfl_xor_sync(0xffffffffu, Mr, o));
    double term = (M0 > -INFINITY ? S0 * (double)ex2f(M0 - Mr) : 0.0) + (M1 > -INFINITY ? S1 * (double)ex2f(M1 - Mr) : 0.0);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) term += __shfl_xor_sync(0xffffffffu, term, o);
    const double lse = ((double)Mr + fast_log2(term)) * 0.69314718055994530942;
    if (lane == 0 && !(term > 0.0 && isfinite(lse))) report(st, CAST_ERR_NONFINITE, row);
    __syncwarp();
    // (e) the K children join the pool
    if (lane < K) {
      const unsigned long long key = topk[lane];
      const float val = key_value(key);
      int tok = key_token(key);
      if (key == 0ull || !(val > -INFINITY) || tok < 0 || tok >= p.V) {  // fewer than K finite logits
        report(st, CAST_ERR_NONFINITE, row);
        tok = 0;
      }
      const size_t o = (size_t)b * p.P;
      const int idx = base + r * K + lane;
      p.pool_score[o + idx] = parent_score + ((double)val - lse);
      p.pool_token[o + idx] = tok;
      p.pool_parent[o + idx] = parent;
      p.pool_depth[o + idx] = p.layer;
      p.pool_kept[o + idx] = 0;
    }
  }

  // ---- layer tail
  __syncthreads();
  const int n_tail = tail_width(p, n_prev);
  if (B <= kTailSingleMaxB) {  // the last CTA of the layer ranks and decides, everything in shared memory
    if (!take_ticket(p.layer_ticket, B * n_prev, &s_flag)) return;
    double* vs = reinterpret_cast<double*>(scratch + 16384);  // [B][CAST_MAX_WIDTH] sorted values
    int* stok = reinterpret_cast<int*>(scratch + 24576);      // [B][CAST_MAX_WIDTH] tokens of the sorted nodes
    tail_rank(p, 0, B, n_tail, n_prev, base, scratch, sorted, stok, vs);
    tail_decide<false>(p, ts, B, n_tail, n_prev, base, sorted, stok, vs);
  } else {  // the last CTA of every sequence ranks that sequence; the last of those decides for the batch
    if (!take_ticket(p.seq_ticket + b, n_prev, &s_flag)) return;
    tail_rank(p, b, 1, n_tail, n_prev, base, scratch, p.tail_sorted, p.tail_tok, p.tail_vs);
    // (tail_rank ends with a CTA barrier: the ticket below releases what all threads wrote)
    if (!take_ticket(p.layer_ticket, B, &s_flag)) return;
    tail_decide<true>(p, ts, B, n_tail, n_prev, base, p.tail_sorted, p.tail_tok, p.tail_vs);
  }
}

// ------------------------------------------------------------------ rerank + linearise
struct SelectParams {
  const double* pool_score;
  const int32_t* pool_token;
  const int32_t* pool_parent;
  const int32_t* pool_depth;
  const int32_t* lsort;
  const double* lscore;
  DevState* st;
  int P, Ncap, words, m, pool_mode, enable_dr, per_row;
  double C3;
  DevTable tab;
  double* sel_score;
  double* sel_value;
  int32_t* sel_idx;
  int32_t* tokens;
  int32_t* parent;
  int32_t* depth;
  uint32_t* anc;
  int32_t* pool_idx;
  double* scores;
  int32_t* n_tree;
};

// Phase 1: rank sequence b's pool under (value desc, depth asc, token asc, creation order) and
// publish the best min(pool, m) nodes with their values. The pool is the root plus one sorted list
// per layer (written by the layer tails in exactly that order restricted to the layer), so the rank
// of the k-th node of a list is k plus, for every other list, the number of its nodes that come
// first: a binary search each. Lists are cut to their first m nodes (later ones cannot rank < m).
__device__ __noinline__ void select_rank_phase(const SelectParams& p, int b, unsigned char* smem) {
  __shared__ int lbase[CAST_MAX_DEPTH + 1], llen[CAST_MAX_DEPTH + 1], loff[CAST_MAX_DEPTH + 2];
  double* ls = reinterpret_cast<double*>(smem);  // the lists' values, list l at loff[l]
  const int tid = threadIdx.x, nt = blockDim.x;
  const size_t o = (size_t)b * p.P;
  const int nl = p.st->layers_done + 1;  // lists: depth 0 (the root) .. layers_done
  if (tid < nl) {  // one memory round trip for all lists
    int len = p.pool_mode == 0 ? p.st->layer_n[tid] : p.st->n_hist[tid];
    llen[tid] = len > p.m ? p.m : len;
    lbase[tid] = p.st->layer_base[tid];
  }
  const int peff = p.pool_mode == 0 ? p.st->pool_size : p.st->kept_total;  // (needed further down)
  __syncthreads();
  if (tid == 0) {
    int acc = 0;
    for (int l = 0; l < nl; ++l) {
      loff[l] = acc;
      acc += llen[l];
    }
    loff[nl] = acc;
  }
  __syncthreads();
  const int total = loff[nl];
#pragma unroll 1
  for (int i = tid; i < total; i += nt) {
    int l = 0;
    while (i >= loff[l + 1]) ++l;
    ls[i] = p.lscore[o + lbase[l] + (i - loff[l])];
  }
  __syncthreads();
  const int n_out = min(min(peff, p.m), p.Ncap);
  int half0 = 1;  // first stride of the searches: positions up to 2 half0 - 1 >= the longest list are reachable
  while (2 * half0 - 1 < p.m && half0 < CAST_MAX_TREE) half0 <<= 1;
#pragma unroll 1
  for (int i = tid; i < total; i += nt) {
    int l = 0;
    while (i >= loff[l + 1]) ++l;
    const int k = i - loff[l];
    const double s = ls[i];
    int rank = k;
    // nodes of another list l2 that come first: value > s, or value == s when their depth is smaller.
    // Lower-bound searches, four lists in lockstep and branch-free so that their loads overlap.
#pragma unroll 1
    for (int l0 = 0; l0 < nl; l0 += 4) {
      int pos[4] = {0, 0, 0, 0}, len4[4], off4[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int l2 = l0 + q;
        const bool valid = l2 < nl && l2 != l;
        len4[q] = valid ? llen[l2] : 0;
        off4[q] = valid ? loff[l2] : 0;
      }
#pragma unroll 1
      for (int half = half0; half >= 1; half >>= 1) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int idx = pos[q] + half - 1;
          const bool inb = idx < len4[q];
          const double a = ls[off4[q] + (inb ? idx : 0)];
          const bool first = inb && ((l0 + q < l) ? (a >= s) : (a > s));
          pos[q] += first ? half : 0;
        }
      }
      rank += pos[0] + pos[1] + pos[2] + pos[3];
    }
    if (rank < n_out) {
      p.sel_score[(size_t)b * p.Ncap + rank] = s;
      p.sel_value[(size_t)b * p.Ncap + rank] = fast_exp_neg(s);
      p.sel_idx[(size_t)b * p.Ncap + rank] = p.lsort[o + lbase[l] + k];
    }
  }
}

// Phase 2: batch-mean utility, target-cost ratio, Algorithm 1 -> N; then sequence b's tree.
__device__ __noinline__ void select_finalize_phase(const SelectParams& p, int b, int B) {
  __shared__ double u[CAST_MAX_TREE], c[CAST_MAX_TREE];
  __shared__ int kept[CAST_MAX_TREE], lin_parent[CAST_MAX_TREE];
  __shared__ short lin_of[1 + CAST_MAX_TOP_K + (CAST_MAX_DEPTH - 1) * CAST_MAX_WIDTH * CAST_MAX_TOP_K];
  __shared__ int s_N;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
  const size_t o = (size_t)b * p.P;
  const int pool = p.st->pool_size;
  const int peff = p.pool_mode == 0 ? pool : p.st->kept_total;
  int n = min(min(peff, p.m), p.Ncap);
  if (p.enable_dr && p.tab.Ntab < n) n = p.tab.Ntab;
  if (tid == 0) s_N = 1;
  // u_k = sum_{s<=k} v(s), v(s) = batch mean of the rank-s values (Eq. 1), or this sequence's own
  // rank-s value when every sequence sizes its tree by itself. The means first, a thread per rank with
  // several loads in flight (u doubles as their buffer), then the prefix sums in one warp.
#pragma unroll 1
  for (int s = tid; s < n; s += nt) {
    double a = 0.0;
    if (p.per_row) {
      a = p.sel_value[(size_t)b * p.Ncap + s];
    } else {
#pragma unroll 8
      for (int bb = 0; bb < B; ++bb) a += p.sel_value[(size_t)bb * p.Ncap + s];
      a /= (double)B;
    }
    u[s] = a;
  }
  __syncthreads();
  if (tid < 32) {
    double v[4], run = 0.0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int s = lane * 4 + e;
      run += s < n ? u[s] : 0.0;
      v[e] = run;
    }
    double incl = run;  // inclusive scan of the lane totals
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const double t = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += t;
    }
    const double excl = incl - run;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int s = lane * 4 + e;
      if (s < n) u[s] = excl + v[e];
    }
  }
  if (p.enable_dr) {
    const int g0 = select_grid(p.st->n0, p.tab.L, p.tab.M);
    const double* f = p.tab.fT + (size_t)(g0 - 1) * p.tab.Ntab;
#pragma unroll 1
    for (int k = tid; k < n; k += nt) c[k] = f[k] / f[0];
  }
  __syncthreads();
  int N = n;
  if (p.enable_dr) {
#pragma unroll 1
    for (int j = tid; j < n; j += nt) {
      bool ok = true;
#pragma unroll 1
      for (int i = 0; i < j; ++i)
        if ((u[j] - u[i]) < p.C3 * (c[j] - c[i])) ok = false;
      if (ok) atomicMax(&s_N, j + 1);
    }
    __syncthreads();
    N = s_N;
  }
  // linearise: kept nodes in creation order (ascending pool index)
#pragma unroll 1
  for (int s = tid; s < N; s += nt) kept[s] = p.sel_idx[(size_t)b * p.Ncap + s];
  __syncthreads();
#pragma unroll 1
  for (int s = tid; s < N; s += nt) {
    const int mine = kept[s];
    int t0 = 0, t1 = 0, j = 0;
    for (; j + 2 <= N; j += 2) {
      t0 += (kept[j] < mine);
      t1 += (kept[j + 1] < mine);
    }
    for (; j < N; ++j) t0 += (kept[j] < mine);
    lin_of[mine] = (short)(t0 + t1);
  }
  __syncthreads();
#pragma unroll 1
  for (int s = tid; s < N; s += nt) {
    const int pi = kept[s];
    const int t = lin_of[pi];
    const int pp = p.pool_parent[o + pi];
    const int lp = pp >= 0 ? (int)lin_of[pp] : -1;
    lin_parent[t] = lp;
    const size_t q = (size_t)b * p.Ncap + t;
    p.tokens[q] = p.pool_token[o + pi];
    p.parent[q] = lp;
    p.depth[q] = p.pool_depth[o + pi];
    p.pool_idx[q] = pi;
    if (p.scores) p.scores[q] = p.pool_score[o + pi];
  }
  __syncthreads();
#pragma unroll 1
  for (int t = tid; t < p.Ncap; t += nt) {
    uint32_t w[CAST_MAX_TREE / 32] = {0u, 0u, 0u, 0u};
    const size_t q = (size_t)b * p.Ncap + t;
    if (t < N) {
      int a = t, guard = 0;
      while (a >= 0 && a < N && guard++ <= CAST_MAX_DEPTH + 1) {  // walk to the root, one bit per ancestor
        w[a >> 5] |= 1u << (a & 31);
        a = lin_parent[a];
      }
    } else {
      p.tokens[q] = -1;
      p.parent[q] = -1;
      p.depth[q] = -1;
      p.pool_idx[q] = -1;
      if (p.scores) p.scores[q] = 0.0;
    }
    for (int k = 0; k < p.words; ++k) p.anc[q * p.words + k] = w[k];
  }
  if (tid == 0) {
    p.n_tree[b] = N;
    if (b == 0) p.st->n_tree = N;
  }
}

__global__ void __launch_bounds__(512) select_rank_kernel(const SelectParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  grid_dependency_wait();
  select_rank_phase(p, blockIdx.x, smem);
}
__global__ void __launch_bounds__(512) select_finalize_kernel(const SelectParams p) {
  select_finalize_phase(p, blockIdx.x, gridDim.x);
}
__global__ void __launch_bounds__(512) select_fused_kernel(const SelectParams p) {  // batch 1: one launch
  extern __shared__ __align__(16) unsigned char smem[];
  grid_dependency_wait();
  select_rank_phase(p, 0, smem);
  __syncthreads();
  select_finalize_phase(p, 0, 1);
}

}  // namespace

// ------------------------------------------------------------------ C-ABI
extern "C" cast_status cast_step_begin(cast_ctx* c, int B, const int32_t* root_token, const int32_t* kv_len,
                                       void* stream) {
  if (!c || !root_token || !kv_len || B < 1) return CAST_ERR_INVALID_ARG;
  if (B > c->cfg.max_batch) return CAST_ERR_CAPACITY;
  const bool need = c->cfg.enable_bp || c->cfg.enable_dp || c->cfg.enable_dr;
  auto it = c->tables->find(B);
  if (it != c->tables->end()) {
    c->cur_table = it->second.dev;
  } else {
    if (need) return CAST_ERR_COST_TABLE;
    c->cur_table = DevTable{1, 1, 1 << 30, nullptr, nullptr};
  }
  c->cur_B = B;
  c->next_layer = 1;
  // Nothing is launched here: the first cast_tree_expand of the step reads root_token and kv_len and resets
  // the per-step state in its own kernel (one launch and one dependent round trip fewer per step).
  c->step_root = root_token;
  c->step_kv_len = kv_len;
  c->tree_inputs_fresh = 1;  // a new step: the engine may have moved the lengths (an attention call decodes afresh)
  (void)stream;
  return CAST_OK;
}

extern "C" cast_status cast_tree_expand(cast_ctx* c, int layer, const void* draft_logits, cast_dtype dtype,
                                        int32_t* next_tokens, int32_t* next_parent_row, int32_t* next_count,
                                        void* stream) {
  if (!c || !draft_logits || !next_tokens || !next_parent_row || !next_count) return CAST_ERR_INVALID_ARG;
  if (dtype != CAST_F32 && dtype != CAST_BF16) return CAST_ERR_DTYPE;
  if (c->cur_B < 1 || layer < 1 || layer > c->cfg.max_depth || layer != c->next_layer) return CAST_ERR_INVALID_ARG;
  c->next_layer = layer + 1;
  const int B = c->cur_B, V = c->cfg.vocab;
  const int rows_per_seq = layer == 1 ? 1 : c->W;
  // A logits row is swept by one cluster of 1 to 8 CTAs. A CTA pays for its fixed phases (prologue, chunk
  // result, cluster barrier and row merge when there is more than one chunk: about 2.5 us, 2 without) and
  // about 4 us per pass of kSweepSub logits, whether the pass is full or not; CTAs beyond one per SM queue
  // up (figures fitted to the measured layer times of the benchmark shapes). The chunk count with the smallest estimate wins: few rows get many one-pass chunks (latency), many
  // rows get few chunks of several full passes (throughput).
  const int rows = B * rows_per_seq;
  int nchunks = 1, chunk_elems = (V + 7) / 8 * 8;
  {
    double best = 1e30;
    for (int n = 1; n <= kSweepMaxChunks; ++n) {
      int ce = ((V + n - 1) / n + 7) / 8 * 8;
      if (n > 1 && ce < 2048) break;  // below this a chunk is all overhead
      const int ne = (V + ce - 1) / ce;
      const int passes = (ce + kSweepSub - 1) / kSweepSub;
      const double per_cta = (ne == 1 ? 2.0 : 2.5) + 4.0 * passes;
      // (a launch a little larger than the machine costs a good part of a second round: the few CTAs left over
      // run while the other SMs idle)
      const double queue = (double)rows * ne / c->num_sms;
      const double cost = per_cta * (queue <= 1.0 ? 1.0 : (queue < 1.5 ? 1.5 : queue));
      if (cost < best - 1e-9) {
        best = cost;
        nchunks = ne;
        chunk_elems = ce;
      }
    }
  }

  ExpandParams p;
  p.logits = draft_logits;
  p.V = V; p.K = c->cfg.top_k; p.W = c->W; p.H = c->cfg.max_depth; p.P = c->P; p.layer = layer;
  p.nchunks = nchunks; p.chunk_elems = chunk_elems;
  // every row that can exist is asked for, whether the previous layer kept it or not: worth it while the
  // whole layer is a small part of the L2 cache
  p.prefetch = (double)rows * V * (dtype == CAST_F32 ? 4 : 2) <= 24e6;
  p.pool_score = c->pool_score; p.pool_token = c->pool_token; p.pool_parent = c->pool_parent;
  p.pool_depth = c->pool_depth; p.pool_kept = c->pool_kept; p.retained = c->retained;
  p.lsort = c->lsort; p.lscore = c->lscore;
  p.st = c->state;
  p.layer_ticket = c->layer_ticket;
  p.seq_ticket = c->seq_ticket; p.tail_vs = c->tail_vs; p.tail_sorted = c->tail_sorted; p.tail_tok = c->tail_tok;
  p.fifo_vals = c->fifo_vals; p.fifo_cnt = c->fifo_cnt; p.R = c->cfg.fifo_len;
  p.tab = c->cur_table;
  p.C1 = c->cfg.C1; p.C2 = c->cfg.C2;
  p.enable_bp = c->cfg.enable_bp; p.enable_dp = c->cfg.enable_dp; p.ctx_base_mode = c->cfg.ctx_base_mode;
  p.next_tokens = next_tokens; p.next_parent_row = next_parent_row; p.next_count = next_count;
  p.root_token = c->step_root; p.kv_len = c->step_kv_len;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(nchunks, rows_per_seq, B);
  cfg.blockDim = dim3(kSweepThreads, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = (cudaStream_t)stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)nchunks;  // the chunks of one row
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // may start before the previous kernel of the stream has drained (the kernel waits where it must)
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const bool queued = (long long)rows * nchunks > c->num_sms;
  cudaError_t e;
  if (dtype == CAST_F32)
    e = queued ? cudaLaunchKernelEx(&cfg, expand_kernel<float, 2>, p) : cudaLaunchKernelEx(&cfg, expand_kernel<float, 1>, p);
  else
    e = queued ? cudaLaunchKernelEx(&cfg, expand_kernel<__nv_bfloat16, 2>, p)
               : cudaLaunchKernelEx(&cfg, expand_kernel<__nv_bfloat16, 1>, p);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return CAST_ERR_CUDA;
  }
  return CAST_OK;
}

extern "C" cast_status cast_select_nodes(cast_ctx* c, int32_t* tokens, int32_t* parent, int32_t* depth,
                                         uint32_t* anc_mask, int32_t* pool_idx, double* scores, int32_t* n_tree,
                                         void* stream) {
  if (!c || !tokens || !parent || !depth || !anc_mask || !pool_idx || !n_tree) return CAST_ERR_INVALID_ARG;
  if (c->cur_B < 1 || c->next_layer < 2) return CAST_ERR_INVALID_ARG;  // a step with at least one layer
  c->tree_inputs_fresh = 1;  // n_tree and the masks: the next attention call reads them after its dependency wait
  SelectParams p;
  p.pool_score = c->pool_score; p.pool_token = c->pool_token; p.pool_parent = c->pool_parent;
  p.pool_depth = c->pool_depth; p.lsort = c->lsort; p.lscore = c->lscore; p.st = c->state;
  p.P = c->P;
  p.Ncap = c->cfg.max_tree; p.words = c->words; p.m = c->cfg.total_token;
  p.pool_mode = c->cfg.pool_mode; p.enable_dr = c->cfg.enable_dr; p.C3 = c->cfg.C3;
  p.per_row = c->cfg.enable_dr && c->cfg.rerank_per_row;
  p.tab = c->cur_table;
  p.sel_score = c->sel_score; p.sel_value = c->sel_value; p.sel_idx = c->sel_idx;
  p.tokens = tokens; p.parent = parent; p.depth = depth; p.anc = anc_mask; p.pool_idx = pool_idx;
  p.scores = scores; p.n_tree = n_tree;
  // the lists' values: (H + 1) lists of at most m nodes
  const size_t smem = (size_t)(c->cfg.max_depth + 1) * c->cfg.total_token * sizeof(double);
  cudaStream_t s = (cudaStream_t)stream;
  int threads = ((c->cfg.max_depth + 1) * c->cfg.total_token + 31) / 32 * 32;
  threads = threads > 512 ? 512 : (threads < 128 ? 128 : threads);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(c->cur_B, 1, 1);
  cfg.blockDim = dim3(threads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see cast_tree_expand
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (c->cur_B == 1) {
    if (cudaLaunchKernelEx(&cfg, select_fused_kernel, p) != cudaSuccess) {
      cudaGetLastError();
      return CAST_ERR_CUDA;
    }
  } else {
    if (cudaLaunchKernelEx(&cfg, select_rank_kernel, p) != cudaSuccess) {
      cudaGetLastError();
      return CAST_ERR_CUDA;
    }
    select_finalize_kernel<<<c->cur_B, 128, 0, s>>>(p);
  }
  return launch_status();
}
