// cast_accept_stochastic: acceptance at temperature T > 0 (Sec. "Speculative Decoding": a draft token with
// draft probability q and target probability p is accepted iff u <= min(1, p/q); after a rejection the
// target distribution is replaced by the residual norm(max(0, P_T - P_D))), walked over the draft tree.
//
// One thread-block cluster per sequence walks the accepted path. At a node every CTA of the cluster holds a
// contiguous slice of the vocabulary: it reads its slice of the node's target and draft logits once, keeps
// exp(logit / T - slice maximum) of both rows in shared memory as fp64, and the cluster agrees on maxima and
// sums through distributed shared memory. The j-th residual has the closed form
//     P_j(x) = max(0, P_T(x) - a_j P_D(x)) / F_j,   a_0 = 0, F_0 = 1, a_{j+1} = a_j + F_j, F_j = F(a_j),
//     F(a) = sum_x max(0, P_T(x) - a P_D(x)),
// (by induction: max(0, max(0, s - a q)/F - q) = max(0, s - (a + F) q)/F), so a rejection costs one sweep
// over the cached slices plus one cluster-wide sum, and the test of a child x is
//     u * P_D(x) * F_j <= max(0, P_T(x) - a_j P_D(x)).
// All arithmetic is fp64: the bonus token is an inverse-CDF sample over up to 150k tokens, where fp32
// rounding would move the result in about one draw of a hundred.
// Every CTA of a cluster computes the same decisions from the same numbers (sums are taken in rank order),
// so the control flow, and with it the sequence of cluster barriers, is uniform across the cluster.
#include <math.h>

#include "cast_internal.h"

using namespace cast;

namespace {

constexpr int kStoThreads = 512;
constexpr int kStoWarps = kStoThreads / 32;
constexpr int kStoMaxCluster = 16;
constexpr int kStoMaxSlice = 12288;  // vocabulary entries a CTA can cache: 2 rows x 8 B each = 192 KB

struct StoParams {
  const void* target_logits;
  const void* draft_logits;
  int V, Ncap, max_depth, slice, cs;
  double inv_T;
  const int32_t* tokens;
  const int32_t* parent;
  const int32_t* n_tree;
  const double* u_accept;
  const double* u_bonus;
  int32_t* accept_len;
  int32_t* accept_path;
  int32_t* bonus_token;
  DevState* st;
};

__device__ __forceinline__ uint32_t sto_smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void sto_st_remote_f64(const double* local, uint32_t rank, double v) {
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(sto_smem_addr(local)), "r"(rank));
  asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(ra), "d"(v) : "memory");
}
__device__ __forceinline__ void sto_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// exp(x) for x <= 0 in fp64 to about 3e-16 relative: x = n ln2 + r with n = round(x log2 e) (ln2 split in
// two so that n ln2_hi is exact), the degree-12 Taylor polynomial of e^r on |r| <= ln2 / 2 (remainder below
// 2e-16), scaling by 2^n through the exponent field. Arguments below -708 (results near the subnormal
// range) give 0; NaN gives NaN. Half the instructions of the general-purpose library routine, and the
// sweeps below are bound by fp64 issue.
__device__ __forceinline__ double sto_exp(double x) {
  // branch-free (a select at the end), so that the compiler can interleave several calls: one call is a
  // chain of some twenty dependent fp64 instructions
  const double xin = x;
  x = fmax(x, -708.0);
  const double kMagic = 6755399441055744.0;  // 1.5 * 2^52: adding it rounds to an integer in the low word
  const double tn = fma(x, 1.4426950408889634074, kMagic);
  const int n = __double2loint(tn);
  const double nd = tn - kMagic;
  double r = fma(nd, -6.93147180369123816490e-01, x);
  r = fma(nd, -1.90821492927058770002e-10, r);
  double y = 2.08767569878680989792e-09;  // 1/12!
  y = fma(y, r, 2.50521083854417187751e-08);
  y = fma(y, r, 2.75573192239858906526e-07);
  y = fma(y, r, 2.75573192239858906526e-06);
  y = fma(y, r, 2.48015873015873015873e-05);
  y = fma(y, r, 1.98412698412698412698e-04);
  y = fma(y, r, 1.38888888888888888889e-03);
  y = fma(y, r, 8.33333333333333333333e-03);
  y = fma(y, r, 4.16666666666666666667e-02);
  y = fma(y, r, 1.66666666666666666667e-01);
  y = fma(y, r, 0.5);
  y = fma(y, r, 1.0);
  y = fma(y, r, 1.0);
  const double res = __hiloint2double(__double2hiint(y) + n * 1048576, __double2loint(y));
  return xin >= -708.0 ? res : (xin != xin ? xin : 0.0);
}

// The same to the same accuracy in half the fp64 instructions, for the pass that evaluates 2 V / cluster-size
// exponentials per node: x = (128 n + j) ln2/128 + r, |r| <= ln2/256, e^x = 2^n * tab[j] * (degree-5 Taylor
// polynomial of e^r, remainder below 1e-18), tab[j] = 2^(j/128) from shared memory.
__device__ __forceinline__ double sto_exp_tab(double x, const double* tab) {
  const double xin = x;
  x = fmax(x, -708.0);
  const double kMagic = 6755399441055744.0;
  const double tn = fma(x, 128.0 * 1.4426950408889634074, kMagic);
  const int k = __double2loint(tn);  // round(x * 128 / ln2), negative or zero
  const double kd = tn - kMagic;
  double r = fma(kd, -6.93147180369123816490e-01 / 128.0, x);
  r = fma(kd, -1.90821492927058770002e-10 / 128.0, r);
  double y = 8.33333333333333333333e-03;
  y = fma(y, r, 4.16666666666666666667e-02);
  y = fma(y, r, 1.66666666666666666667e-01);
  y = fma(y, r, 0.5);
  y = fma(y, r, 1.0);
  y = fma(y, r, 1.0);
  y *= tab[k & 127];
  const double res = __hiloint2double(__double2hiint(y) + (k >> 7) * 1048576, __double2loint(y));
  return xin >= -708.0 ? res : (xin != xin ? xin : 0.0);
}

struct StoShared {
  double xch[2][kStoMaxCluster][4];  // records of the cluster's CTAs, double-buffered by exchange parity
  double wred[kStoWarps][4];
  int32_t par[CAST_MAX_TREE];
  int32_t tok[CAST_MAX_TREE];
  int32_t kids[CAST_MAX_TREE];
  int32_t nkids;
  int32_t pick_lo, pick_hi;
  double wscan[kStoWarps];
  double tab[128];  // 2^(j/128)
};

// Block-wide reduction of up to four values per thread (sum, or maximum for OP_MAX); every thread returns
// with the result, folded in warp order.
template <bool OP_MAX, int NVAL>
__device__ __forceinline__ void sto_block_reduce(StoShared& sh, double (&v)[NVAL]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < NVAL; ++i) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double other = __shfl_xor_sync(0xffffffffu, v[i], o);
      v[i] = OP_MAX ? fmax(v[i], other) : v[i] + other;
    }
  }
  __syncthreads();  // the previous reduction's readers are done with wred
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < NVAL; ++i) sh.wred[warp][i] = v[i];
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < NVAL; ++i) {
    double acc = sh.wred[0][i];
#pragma unroll
    for (int w = 1; w < kStoWarps; ++w) acc = OP_MAX ? fmax(acc, sh.wred[w][i]) : acc + sh.wred[w][i];
    v[i] = acc;
  }
}

// Every CTA hands its record to every CTA of the cluster (its own copy included); after the barrier
// sh.xch[parity][r] holds rank r's record everywhere.
__device__ __forceinline__ void sto_exchange(StoShared& sh, int parity, int rank, int cs, const double (&rec)[4]) {
  if (cs == 1) {
    __syncthreads();
    if (threadIdx.x < 4) sh.xch[parity][0][threadIdx.x] = rec[threadIdx.x];
    __syncthreads();
    return;
  }
  const int tid = threadIdx.x;
  if (tid < cs * 4) sto_st_remote_f64(&sh.xch[parity][rank][tid & 3], (uint32_t)(tid >> 2), rec[tid & 3]);
  sto_cluster_sync();
}

template <typename T, bool CACHED>
__global__ void __launch_bounds__(kStoThreads, 1) accept_stochastic_kernel(const StoParams p) {
  extern __shared__ __align__(16) unsigned char sto_dyn[];
  __shared__ StoShared sh;
  double* ep = reinterpret_cast<double*>(sto_dyn);  // exp(target logit / T - slice maximum), this CTA's slice
  double* eq = ep + p.slice;                        // the same of the draft row
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cs = p.cs, rank = blockIdx.x, b = blockIdx.y;
  const int begin = min(rank * p.slice, p.V), len = min(p.V - begin, p.slice);
  int N = p.n_tree[b];
  if (N < 1 || N > p.Ncap) {
    if (rank == 0 && tid == 0) report(p.st, CAST_ERR_BAD_TREE, b);
    N = N < 1 ? 1 : p.Ncap;
  }
  if (tid >= kStoThreads - 128) sh.tab[tid - (kStoThreads - 128)] = exp2((double)(tid - (kStoThreads - 128)) * (1.0 / 128.0));
  if (tid < CAST_MAX_TREE) {
    sh.par[tid] = tid < N ? p.parent[(size_t)b * p.Ncap + tid] : -2;
    sh.tok[tid] = tid < N ? p.tokens[(size_t)b * p.Ncap + tid] : 0;
  }
  // the peers' shared memory may be written once all CTAs of the cluster run
  if (cs > 1) sto_cluster_sync(); else __syncthreads();

  int parity = 0;
  int cur = 0, plen = 1;   // current node, nodes on the path so far
  double a = 0.0;          // the distribution that stands at `cur`: max(0, P_T - a P_D) / F(a)
  double cp = 0.0, cq = 0.0, Mp = 0.0, Sp = 1.0, Mq = 0.0, Sq = 1.0, Mp_loc = 0.0, Mq_loc = 0.0;
  const T* lp = nullptr;
  const T* lq = nullptr;
  bool has_q = false;
  if (rank == 0 && tid == 0) p.accept_path[(size_t)b * (p.max_depth + 1)] = 0;

  // unnormalised slice entries: p~(i) * cp = P_T(begin + i), q~(i) * cq = P_D(begin + i)
  auto pt = [&](int i) -> double {
    return CACHED ? ep[i] : sto_exp_tab((double)to_float(lp[begin + i]) * p.inv_T - (Mp_loc > -INFINITY ? Mp_loc : 0.0), sh.tab);
  };
  auto qt = [&](int i) -> double {
    return CACHED ? eq[i] : sto_exp_tab((double)to_float(lq[begin + i]) * p.inv_T - (Mq_loc > -INFINITY ? Mq_loc : 0.0), sh.tab);
  };

  for (;;) {
    // ---- children of `cur` in tree order
    __syncthreads();  // everybody is done with the previous node's list
    if (warp == 0) {
      int n = 0;
      for (int base = 0; base < N; base += 32) {
        const int c = base + lane;
        const bool is = c < N && c > cur && sh.par[c] == cur;
        const unsigned m = __ballot_sync(0xffffffffu, is);
        if (is) sh.kids[n + __popc(m & ((1u << lane) - 1u))] = c;
        n += __popc(m);
      }
      if (lane == 0) sh.nkids = n;
    }
    __syncthreads();
    int k = sh.nkids;
    if (k > 0 && plen > p.max_depth) {  // a path longer than the output has room for
      if (rank == 0 && tid == 0) report(p.st, CAST_ERR_BAD_TREE, b);
      k = 0;
    }
    has_q = k > 0;
    lp = reinterpret_cast<const T*>(p.target_logits) + ((size_t)b * p.Ncap + cur) * p.V;
    lq = reinterpret_cast<const T*>(p.draft_logits) + ((size_t)b * p.Ncap + cur) * p.V;
    if (k > 0) {
      // the eldest child is the likeliest next node: its slices are asked into L2 while this node is worked on
      const int c0 = sh.kids[0];
      const char* np = reinterpret_cast<const char*>(reinterpret_cast<const T*>(p.target_logits) + ((size_t)b * p.Ncap + c0) * p.V + begin);
      const char* nq = reinterpret_cast<const char*>(reinterpret_cast<const T*>(p.draft_logits) + ((size_t)b * p.Ncap + c0) * p.V + begin);
      for (int off = tid * 128; off < len * (int)sizeof(T); off += kStoThreads * 128) {
        asm volatile("prefetch.global.L2 [%0];" ::"l"(np + off));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(nq + off));
      }
    }

    // the eldest child's test needs two logits and its uniform number: asked for now, used after the sweeps
    float raw0 = 0.f;
    double u0 = 0.0;
    if (k > 0) {
      const int c0 = sh.kids[0], x0 = sh.tok[c0];
      if (x0 >= 0 && x0 < p.V) raw0 = (lane & 1) ? to_float(lq[x0]) : to_float(lp[x0]);
      u0 = p.u_accept[(size_t)b * p.Ncap + c0];
    }

    // ---- softmax statistics of the node's rows: slice maxima, then slice sums of exp(. - slice maximum)
    {
      double mx[2] = {-INFINITY, -INFINITY};
#pragma unroll 8
      for (int i = tid; i < len; i += kStoThreads) {
        const double sp = (double)to_float(lp[begin + i]) * p.inv_T;
        if (CACHED) ep[i] = sp;
        mx[0] = fmax(mx[0], sp);
        if (has_q) {
          const double sq = (double)to_float(lq[begin + i]) * p.inv_T;
          if (CACHED) eq[i] = sq;
          mx[1] = fmax(mx[1], sq);
        }
      }
      sto_block_reduce<true, 2>(sh, mx);
      Mp_loc = mx[0];
      Mq_loc = mx[1];
      double sm[2] = {0.0, 0.0};
      // an all -inf slice (a masked range of the vocabulary) takes reference 0: its entries become exp(-inf) = 0
      const double ref_p = Mp_loc > -INFINITY ? Mp_loc : 0.0, ref_q = Mq_loc > -INFINITY ? Mq_loc : 0.0;
      if (has_q) {
#pragma unroll 4
        for (int i = tid; i < len; i += kStoThreads) {
          const double e0 = sto_exp_tab((CACHED ? ep[i] : (double)to_float(lp[begin + i]) * p.inv_T) - ref_p, sh.tab);
          const double e1 = sto_exp_tab((CACHED ? eq[i] : (double)to_float(lq[begin + i]) * p.inv_T) - ref_q, sh.tab);
          if (CACHED) {
            ep[i] = e0;
            eq[i] = e1;
          }
          sm[0] += e0;
          sm[1] += e1;
        }
      } else {
#pragma unroll 4
        for (int i = tid; i < len; i += kStoThreads) {
          const double e0 = sto_exp_tab((CACHED ? ep[i] : (double)to_float(lp[begin + i]) * p.inv_T) - ref_p, sh.tab);
          if (CACHED) ep[i] = e0;
          sm[0] += e0;
        }
      }
      sto_block_reduce<false, 2>(sh, sm);
      const double rec[4] = {Mp_loc, sm[0], Mq_loc, sm[1]};
      sto_exchange(sh, parity, rank, cs, rec);
      // fold of the ranks' records, the same in every warp of every CTA: lanes 0-15 take the target row's
      // records by rank, lanes 16-31 the draft row's; maxima and sums through a fixed shuffle tree
      {
        const int rr = lane & 15, col = (lane >> 4) * 2;
        const double m_r = rr < cs ? sh.xch[parity][rr][col] : -INFINITY;
        const double s_r = rr < cs ? sh.xch[parity][rr][col + 1] : 0.0;
        double M = m_r;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) M = fmax(M, __shfl_xor_sync(0xffffffffu, M, o));
        const double w_r = m_r > -INFINITY ? sto_exp(m_r - M) : 0.0;  // this rank's weight
        double S = s_r * w_r;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) S += __shfl_xor_sync(0xffffffffu, S, o);
        Mp = __shfl_sync(0xffffffffu, M, 0);
        Mq = __shfl_sync(0xffffffffu, M, 16);
        Sp = __shfl_sync(0xffffffffu, S, 0);
        Sq = __shfl_sync(0xffffffffu, S, 16);
        cp = __shfl_sync(0xffffffffu, w_r, rank);        // exp(Mp_loc - Mp)
        cq = __shfl_sync(0xffffffffu, w_r, 16 + rank);   // exp(Mq_loc - Mq)
      }
      parity ^= 1;
      if (!(Sp > 0.0) || !isfinite(Sp) || (has_q && (!(Sq > 0.0) || !isfinite(Sq)))) {
        if (rank == 0 && tid == 0) report(p.st, CAST_ERR_NONFINITE, b * p.Ncap + cur);
        Sp = 1.0;  // keep the arithmetic finite; the result of this sequence is void
        Sq = 1.0;
        k = 0;
        has_q = false;
      }
      cp = cp / Sp;
      cq = has_q ? cq / Sq : 0.0;
    }

    // ---- the children, one after the other, each against the residual its elder siblings left
    a = 0.0;
    double F = 1.0;
    int next = -1;
    for (int j = 0; j < k; ++j) {
      const int c = sh.kids[j];
      const int x = sh.tok[c];
      if (x < 0 || x >= p.V) {
        if (rank == 0 && tid == 0) report(p.st, CAST_ERR_BAD_TREE, b);
        continue;  // not a token: never accepted
      }
      const double u = j == 0 ? u0 : p.u_accept[(size_t)b * p.Ncap + c];
      const float raw = j == 0 ? raw0 : ((lane & 1) ? to_float(lq[x]) : to_float(lp[x]));  // odd lanes: draft
      const double v01 = (lane & 1) ? sto_exp((double)raw * p.inv_T - Mq) / Sq : sto_exp((double)raw * p.inv_T - Mp) / Sp;
      const double px = __shfl_sync(0xffffffffu, v01, 0), qx = __shfl_sync(0xffffffffu, v01, 1);
      const double rx = fmax(0.0, px - a * qx);
      if (u * qx * F <= rx) {
        next = c;
        break;
      }
      // rejected: the residual of the residual
      const double a2 = a + F;
      double part[1] = {0.0};
#pragma unroll 4
      for (int i = tid; i < len; i += kStoThreads) part[0] += fmax(0.0, pt(i) * cp - a2 * (qt(i) * cq));
      sto_block_reduce<false, 1>(sh, part);
      const double rec[4] = {part[0], 0.0, 0.0, 0.0};
      sto_exchange(sh, parity, rank, cs, rec);
      double F2 = 0.0;
      for (int r = 0; r < cs; ++r) F2 += sh.xch[parity][r][0];
      parity ^= 1;
      if (!(F2 > 0.0)) break;  // an empty residual: the distribution before it stands
      a = a2;
      F = F2;
    }
    if (next < 0) break;
    cur = next;
    if (rank == 0 && tid == 0) p.accept_path[(size_t)b * (p.max_depth + 1) + plen] = cur;
    ++plen;
  }

  // ---- bonus token: inversion of the cumulative sum, in token order, of max(0, P_T - a P_D) at `cur`
  double part[1] = {0.0};
#pragma unroll 4
  for (int i = tid; i < len; i += kStoThreads) part[0] += fmax(0.0, pt(i) * cp - (has_q ? a * (qt(i) * cq) : 0.0));
  sto_block_reduce<false, 1>(sh, part);
  {
    const double rec[4] = {part[0], 0.0, 0.0, 0.0};
    sto_exchange(sh, parity, rank, cs, rec);
  }
  double total = 0.0;
  for (int r = 0; r < cs; ++r) total += sh.xch[parity][r][0];
  const double goal = p.u_bonus[b] * total;
  // the slice in which the cumulative sum reaches the goal (rounding may leave none: the last non-empty one)
  int owner = -1, last_nonempty = 0;
  double before = 0.0, before_owner = 0.0;
  for (int r = 0; r < cs; ++r) {
    const double s = sh.xch[parity][r][0];
    if (s > 0.0) last_nonempty = r;
    if (owner < 0 && before + s >= goal && s > 0.0) {
      owner = r;
      before_owner = before;
    }
    before += s;
  }
  if (owner < 0) {
    owner = last_nonempty;
    before_owner = 0.0;
    for (int r = 0; r < owner; ++r) before_owner += sh.xch[parity][r][0];
  }
  if (rank == 0 && tid == 0) {
    p.accept_len[b] = plen - 1;
    for (int j = plen; j <= p.max_depth; ++j) p.accept_path[(size_t)b * (p.max_depth + 1) + j] = -1;
  }
  if (rank != owner) return;

  // thread t owns the contiguous piece [t * seg, (t + 1) * seg) of the slice
  const int seg = (len + kStoThreads - 1) / kStoThreads;
  const int i0 = min(tid * seg, len), i1 = min(i0 + seg, len);
  const double qa = has_q ? a : 0.0;
  double mine = 0.0;
  for (int i = i0; i < i1; ++i) mine += fmax(0.0, pt(i) * cp - (has_q ? qa * (qt(i) * cq) : 0.0));
  double incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double other = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += other;
  }
  if (tid == 0) {
    sh.pick_lo = kStoThreads;
    sh.pick_hi = -1;
  }
  __syncthreads();
  if (lane == 31) sh.wscan[warp] = incl;
  __syncthreads();
  double offs = before_owner;
  for (int w = 0; w < warp; ++w) offs += sh.wscan[w];
  incl += offs;
  const double excl = incl - mine;
  if (mine > 0.0) {
    atomicMax(&sh.pick_hi, tid);
    if (incl >= goal) atomicMin(&sh.pick_lo, tid);
  }
  __syncthreads();
  const int pick = sh.pick_lo < kStoThreads ? sh.pick_lo : sh.pick_hi;
  if (pick < 0) {  // nothing has mass here (a void sequence): token 0
    if (tid == 0) p.bonus_token[b] = 0;
    return;
  }
  if (tid == pick) {
    double run = excl;
    int tokx = -1, last = i0;
    for (int i = i0; i < i1; ++i) {
      const double r = fmax(0.0, pt(i) * cp - (has_q ? qa * (qt(i) * cq) : 0.0));
      if (r > 0.0) last = i;
      run += r;
      if (run >= goal && r > 0.0) {
        tokx = i;
        break;
      }
    }
    p.bonus_token[b] = begin + (tokx >= 0 ? tokx : last);
  }
}

template <typename T, bool CACHED>
cast_status sto_launch(const StoParams& p, int B, size_t dyn, cudaStream_t s) {
  auto kern = accept_stochastic_kernel<T, CACHED>;
  CAST_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn));
  if (p.cs > 8) CAST_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.cs, B, 1);
  cfg.blockDim = dim3(kStoThreads, 1, 1);
  cfg.dynamicSmemBytes = dyn;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = p.cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  CAST_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, p));
  return CAST_OK;
}

// Largest cluster size (16, else 8) with which a CTA of `dyn` bytes of dynamic shared memory can run.
template <typename T, bool CACHED>
int sto_max_cluster(size_t dyn16, size_t dyn8) {
  auto kern = accept_stochastic_kernel<T, CACHED>;
  for (int cs = 16; cs >= 8; cs >>= 1) {
    const size_t dyn = cs == 16 ? dyn16 : dyn8;
    if (dyn > (size_t)kStoMaxSlice * 16) continue;  // this slice does not fit
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess ||
        (cs > 8 && cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)) {
      (void)cudaGetLastError();
      continue;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cs, 1, 1);
    cfg.blockDim = dim3(kStoThreads, 1, 1);
    cfg.dynamicSmemBytes = dyn;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) == cudaSuccess && n >= 1) return cs;
    (void)cudaGetLastError();
  }
  (void)cudaGetLastError();
  return 0;
}

int slice_for(int V, int cs) { return ((V + cs - 1) / cs + 7) / 8 * 8; }

}  // namespace

namespace {
// Cluster size and caching mode for this context's vocabulary and a logits dtype, looked up once.
void sto_plan(cast_ctx* c, bool f32) {
  const int di = f32 ? 0 : 1;
  if (c->sto_cs[di] != 0) return;
  const int V = c->cfg.vocab;
  const size_t d16 = (size_t)slice_for(V, 16) * 16, d8 = (size_t)slice_for(V, 8) * 16;
  int cs = f32 ? sto_max_cluster<float, true>(d16, d8) : sto_max_cluster<__nv_bfloat16, true>(d16, d8);
  int cached = 1;
  if (cs == 0) {
    cached = 0;
    cs = f32 ? sto_max_cluster<float, false>(0, 0) : sto_max_cluster<__nv_bfloat16, false>(0, 0);
    if (cs == 0) cs = 1;
  }
  c->sto_cs[di] = cs;
  c->sto_cached[di] = cached;
}
}  // namespace

extern "C" cast_status cast_accept_stochastic_plan(cast_ctx* c, cast_dtype dtype, int* cluster_size, int* cached) {
  if (!c || !cluster_size || !cached) return CAST_ERR_INVALID_ARG;
  if (dtype != CAST_F32 && dtype != CAST_BF16) return CAST_ERR_DTYPE;
  sto_plan(c, dtype == CAST_F32);
  *cluster_size = c->sto_cs[dtype == CAST_F32 ? 0 : 1];
  *cached = c->sto_cached[dtype == CAST_F32 ? 0 : 1];
  return CAST_OK;
}

extern "C" cast_status cast_accept_stochastic(cast_ctx* c, const void* target_logits, const void* draft_logits,
                                              cast_dtype dtype, int B, double temperature, const int32_t* tokens,
                                              const int32_t* parent, const int32_t* n_tree, const double* u_accept,
                                              const double* u_bonus, int32_t* accept_len, int32_t* accept_path,
                                              int32_t* bonus_token, void* stream) {
  if (!c || !target_logits || !draft_logits || !tokens || !parent || !n_tree || !u_accept || !u_bonus || !accept_len ||
      !accept_path || !bonus_token || B < 1 || !(temperature > 0.0) || !isfinite(temperature))
    return CAST_ERR_INVALID_ARG;
  if (dtype != CAST_F32 && dtype != CAST_BF16) return CAST_ERR_DTYPE;
  if (B > c->cfg.max_batch) return CAST_ERR_CAPACITY;
  const int V = c->cfg.vocab;
  // cluster size: 16 CTAs per sequence where the device can co-schedule them, else 8; the slices are cached
  // in shared memory when they fit, else every sweep recomputes them from the logits
  const bool f32 = dtype == CAST_F32;
  const int di = f32 ? 0 : 1;
  sto_plan(c, f32);  // first call with this dtype: a host-side query, no device work
  const int cs = c->sto_cs[di];
  const bool cached = c->sto_cached[di] != 0;
  StoParams p;
  p.target_logits = target_logits;
  p.draft_logits = draft_logits;
  p.V = V;
  p.Ncap = c->cfg.max_tree;
  p.max_depth = c->cfg.max_depth;
  p.cs = cs;
  p.slice = slice_for(V, cs);
  p.inv_T = 1.0 / temperature;
  p.tokens = tokens;
  p.parent = parent;
  p.n_tree = n_tree;
  p.u_accept = u_accept;
  p.u_bonus = u_bonus;
  p.accept_len = accept_len;
  p.accept_path = accept_path;
  p.bonus_token = bonus_token;
  p.st = c->state;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t dyn = cached ? (size_t)p.slice * 16 : 0;
  if (f32) return cached ? sto_launch<float, true>(p, B, dyn, s) : sto_launch<float, false>(p, B, dyn, s);
  return cached ? sto_launch<__nv_bfloat16, true>(p, B, dyn, s) : sto_launch<__nv_bfloat16, false>(p, B, dyn, s);
}
