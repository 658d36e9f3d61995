// cast_tree_attention: tree-masked verification attention.
//
// CUDA-core path (fp32 inputs, and any shape the tensor-core path does not take): a
// flash-style kernel. One CTA owns (sequence, kv-head, block of 32 query rows, KV split); a
// query row is a (tree token, head of the GQA group) pair, so a K/V tile fetched once serves
// all tree tokens and all heads of the group. Tiles of 64 positions are converted to fp32 in
// shared memory; S = QK^T and O += PV are register-tiled FFMA loops; the softmax is online.
// Prefix positions need no mask; a tree position L+j is visible to row (t, g) iff bit j of
// anc_mask[t] is set. KV splits write (max, sum, unnormalised O) partials that a second
// kernel merges.
#include <math.h>

#include "cast_internal.h"

using namespace cast;

namespace cast {
// implemented in tree_attention_tc.cu; returns false when the shape is not taken there
bool tree_attention_tc_launch(cast_ctx* c, const void* q, const void* k, const void* v, int B, int Hq, int Hkv, int D,
                              int page_size, const int32_t* page_table, int seq_capacity, int num_pages,
                              const int32_t* kv_len, const uint32_t* anc, const int32_t* n_tree, const int32_t* first_row,
                              float scale, void* out, cudaStream_t stream, cast_status* status);
size_t tree_attention_tc_workspace(const cast_ctx* c, int B, int Hq, int Hkv, int D, int page_size, int seq_capacity);
cast_status tree_attention_tc_reserve(cast_ctx* c, size_t bytes);
}

namespace {

constexpr int kRB = 32;   // query rows per CTA
constexpr int kPT = 64;   // positions per tile
constexpr int kThreads = 256;
constexpr int kMaxSplit = 64;

struct AttnParams {
  const void* q;
  const void* k;
  const void* v;
  void* out;
  int B, Ncap, Hq, Hkv, G, page_size, seq_capacity, num_pages, words, nsplit;
  const int32_t* page_table;
  const int32_t* kv_len;
  const int32_t* n_tree;
  const int32_t* first_row;  // [B] or null: output rows start at this tree token
  const uint32_t* anc;
  float scale;
  float* part_o;   // [B][Hq][Ncap][nsplit][D]
  float* part_ml;  // [B][Hq][Ncap][nsplit][2]
  DevState* st;
};

template <typename T> __device__ __forceinline__ void load_chunk(const T* p, float* out);
template <> __device__ __forceinline__ void load_chunk<float>(const float* p, float* out) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
}
template <> __device__ __forceinline__ void load_chunk<__nv_bfloat16>(const __nv_bfloat16* p, float* out) {
  const uint4 a = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void store_out(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) tree_attn_cc_kernel(const AttnParams p) {
  constexpr int KS = D + 4;          // padded row stride of Qs / Ks (floats)
  constexpr int SS = kPT + 1;        // row stride of Ss
  constexpr int CH = 16 / sizeof(T); // elements per 16-byte chunk
  constexpr int CPR = D / CH;        // chunks per cache row
  constexpr int DC = D / 32;         // output columns per lane
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;                       // [kRB][KS]
  float* Ks = Qs + kRB * KS;              // [kPT][KS]
  float* Vs = Ks + kPT * KS;              // [kPT][D]
  float* Ss = Vs + kPT * D;               // [kRB][SS]
  __shared__ float row_m[kRB], row_l[kRB], row_alpha[kRB];
  __shared__ uint32_t anc_s[kRB][CAST_MAX_TREE / 32];
  __shared__ long long slot_s[kPT];

  const int split = blockIdx.x % p.nsplit, rb = blockIdx.x / p.nsplit;
  const int kvh = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int N = p.n_tree[b];
  N = N < 0 ? 0 : (N > p.Ncap ? p.Ncap : N);
  int L = p.kv_len[b];
  if (L < 0) L = 0;
  const int G = p.G;
  int F = p.first_row != nullptr ? p.first_row[b] : 0;  // tokens before F are context only
  F = F < 0 ? 0 : (F > N ? N : F);
  const int rows_total = (N - F) * G;
  const int row0 = rb * kRB;
  if (row0 >= rows_total) return;
  const int max_pos = p.page_size == 0 ? p.seq_capacity : p.seq_capacity * p.page_size;
  int total = L + N;
  if (total > max_pos) {
    if (tid == 0) report(p.st, CAST_ERR_BAD_PAGE, b);
    total = max_pos;
  }
  const int ntiles = (total + kPT - 1) / kPT;
  const int t0 = (int)((long long)split * ntiles / p.nsplit), t1 = (int)((long long)(split + 1) * ntiles / p.nsplit);

  // query rows (pre-scaled), their ancestor masks, running softmax state
  const T* q = reinterpret_cast<const T*>(p.q);
  for (int i = tid; i < kRB * CPR; i += kThreads) {
    const int r = i / CPR, ch = i % CPR, row = row0 + r;
    float f[CH];
    if (row < rows_total) {
      const int t = F + row / G, g = row % G;
      load_chunk<T>(q + (((size_t)b * p.Ncap + t) * p.Hq + kvh * G + g) * D + ch * CH, f);
    } else {
#pragma unroll
      for (int e = 0; e < CH; ++e) f[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < CH; ++e) Qs[r * KS + ch * CH + e] = f[e] * p.scale;
  }
  if (tid < kRB) {
    row_m[tid] = -INFINITY;
    row_l[tid] = 0.f;
    const int row = row0 + tid;
    for (int w = 0; w < CAST_MAX_TREE / 32; ++w)
      anc_s[tid][w] = (row < rows_total && w < p.words) ? p.anc[((size_t)b * p.Ncap + F + row / G) * p.words + w] : 0u;
  }
  float o[4][DC];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int e = 0; e < DC; ++e) o[i][e] = 0.f;

  const T* kc = reinterpret_cast<const T*>(p.k);
  const T* vc = reinterpret_cast<const T*>(p.v);
  const int ty = tid / 16, tx = tid % 16;

  for (int tile = t0; tile < t1; ++tile) {
    const int pbase = tile * kPT;
    __syncthreads();  // previous tile fully consumed; Qs/anc_s visible on the first pass
    if (tid < kPT) {
      const int pos = pbase + tid;
      long long slot = -1;
      if (pos < total) {
        if (p.page_size == 0) {
          slot = (long long)b * p.seq_capacity + pos;
        } else {
          const int page = p.page_table[(size_t)b * p.seq_capacity + pos / p.page_size];
          if (page < 0 || page >= p.num_pages) report(p.st, CAST_ERR_BAD_PAGE, b);
          else slot = (long long)page * p.page_size + pos % p.page_size;
        }
      }
      slot_s[tid] = slot;
    }
    __syncthreads();
    for (int i = tid; i < kPT * CPR; i += kThreads) {
      const int pl = i / CPR, ch = i % CPR;
      const long long slot = slot_s[pl];
      float fk[CH], fv[CH];
      if (slot >= 0) {
        const size_t off = ((size_t)slot * p.Hkv + kvh) * D + ch * CH;
        load_chunk<T>(kc + off, fk);
        load_chunk<T>(vc + off, fv);
      } else {
#pragma unroll
        for (int e = 0; e < CH; ++e) fk[e] = fv[e] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < CH; ++e) {
        Ks[pl * KS + ch * CH + e] = fk[e];
        Vs[pl * D + ch * CH + e] = fv[e];
      }
    }
    __syncthreads();
    // S = Q K^T: thread (ty, tx) owns rows 2ty, 2ty+1 and positions tx, tx+16, tx+32, tx+48
    {
      float acc[2][4];
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 8
      for (int d = 0; d < D; d += 4) {
        const float4 q0 = *reinterpret_cast<const float4*>(Qs + (2 * ty) * KS + d);
        const float4 q1 = *reinterpret_cast<const float4*>(Qs + (2 * ty + 1) * KS + d);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float4 kk = *reinterpret_cast<const float4*>(Ks + (tx + 16 * j) * KS + d);
          acc[0][j] += q0.x * kk.x + q0.y * kk.y + q0.z * kk.z + q0.w * kk.w;
          acc[1][j] += q1.x * kk.x + q1.y * kk.y + q1.z * kk.z + q1.w * kk.w;
        }
      }
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int r = 2 * ty + i;
        const bool row_ok = row0 + r < rows_total;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int pl = tx + 16 * j, pos = pbase + pl;
          bool vis = row_ok && pos < total;
          if (vis && pos >= L) {
            const int jt = pos - L;
            vis = (anc_s[r][jt >> 5] >> (jt & 31)) & 1u;
          }
          Ss[r * SS + pl] = vis ? acc[i][j] : -INFINITY;
        }
      }
    }
    __syncthreads();
    // online softmax and O += P V: warp w owns rows 4w .. 4w+3
#pragma unroll
    for (int rr = 0; rr < 4; ++rr) {
      const int r = 4 * warp + rr;
      const float s0 = Ss[r * SS + lane], s1 = Ss[r * SS + lane + 32];
      float mx = fmaxf(s0, s1);
#pragma unroll
      for (int of = 16; of > 0; of >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, of));
      const float m_old = row_m[r];
      const float m_new = fmaxf(m_old, mx);
      float p0 = 0.f, p1 = 0.f, alpha = 1.f;
      if (m_new > -INFINITY) {
        p0 = expf(s0 - m_new);
        p1 = expf(s1 - m_new);
        alpha = expf(m_old - m_new);
      }
      float sum = p0 + p1;
#pragma unroll
      for (int of = 16; of > 0; of >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, of);
      __syncwarp();
      Ss[r * SS + lane] = p0;
      Ss[r * SS + lane + 32] = p1;
      if (lane == 0) {
        row_m[r] = m_new;
        row_l[r] = row_l[r] * alpha + sum;
        row_alpha[r] = alpha;
      }
    }
    __syncwarp();
#pragma unroll
    for (int rr = 0; rr < 4; ++rr) {
      const float a = row_alpha[4 * warp + rr];
#pragma unroll
      for (int e = 0; e < DC; ++e) o[rr][e] *= a;
    }
#pragma unroll 4
    for (int pl = 0; pl < kPT; ++pl) {
      float vv[DC];
      if constexpr (DC == 4) {
        const float4 t4 = *reinterpret_cast<const float4*>(Vs + pl * D + lane * 4);
        vv[0] = t4.x; vv[1] = t4.y; vv[2] = t4.z; vv[3] = t4.w;
      } else {
        const float2 t2 = *reinterpret_cast<const float2*>(Vs + pl * D + lane * 2);
        vv[0] = t2.x; vv[1] = t2.y;
      }
#pragma unroll
      for (int rr = 0; rr < 4; ++rr) {
        const float pv = Ss[(4 * warp + rr) * SS + pl];
#pragma unroll
        for (int e = 0; e < DC; ++e) o[rr][e] += pv * vv[e];
      }
    }
  }
  __syncthreads();
  // partials of this split
#pragma unroll
  for (int rr = 0; rr < 4; ++rr) {
    const int r = 4 * warp + rr, row = row0 + r;
    if (row >= rows_total) continue;
    const int t = F + row / G, h = kvh * G + row % G;
    const size_t pr = (((size_t)b * p.Hq + h) * p.Ncap + t) * p.nsplit + split;
#pragma unroll
    for (int e = 0; e < DC; ++e) p.part_o[pr * D + lane * DC + e] = o[rr][e];
    if (lane == 0) {
      p.part_ml[pr * 2] = row_m[r];
      p.part_ml[pr * 2 + 1] = row_l[r];
    }
  }
}

// Merge the split partials of one (sequence, tree token, head); rows >= n_tree are left untouched.
template <typename T, int D>
__global__ void __launch_bounds__(D) attn_combine_kernel(const AttnParams p) {
  const int t = blockIdx.x, h = blockIdx.y, b = blockIdx.z, d = threadIdx.x;
  T* out = reinterpret_cast<T*>(p.out) + (((size_t)b * p.Ncap + t) * p.Hq + h) * D;
  int N = p.n_tree[b];
  N = N > p.Ncap ? p.Ncap : N;
  if (t >= N || (p.first_row != nullptr && t < p.first_row[b])) return;
  const size_t pr = (((size_t)b * p.Hq + h) * p.Ncap + t) * p.nsplit;
  float M = -INFINITY;
  for (int s = 0; s < p.nsplit; ++s) M = fmaxf(M, p.part_ml[(pr + s) * 2]);
  float l = 0.f, acc = 0.f;
  for (int s = 0; s < p.nsplit; ++s) {
    const float ms = p.part_ml[(pr + s) * 2];
    if (ms > -INFINITY) {
      const float w = expf(ms - M);
      l += p.part_ml[(pr + s) * 2 + 1] * w;
      acc += p.part_o[(pr + s) * D + d] * w;
    }
  }
  store_out(out + d, l > 0.f ? acc / l : 0.f);
}

// KV splits of a CUDA-core launch and the partial rows its workspace holds.
int cc_splits(const cast_ctx* c, int B, int Hkv, int G, int page_size, int seq_capacity) {
  const int base = B * Hkv * ((c->cfg.total_token * G + kRB - 1) / kRB);
  int nsplit = (2 * c->num_sms + base - 1) / base;
  const int max_pos = page_size == 0 ? seq_capacity : seq_capacity * page_size;
  const int max_tiles = (max_pos + kPT - 1) / kPT;
  if (nsplit > max_tiles) nsplit = max_tiles;
  if (nsplit > kMaxSplit) nsplit = kMaxSplit;
  if (nsplit < 1) nsplit = 1;
  return nsplit;
}
size_t cc_workspace(const cast_ctx* c, int B, int Hq, int Hkv, int D, int page_size, int seq_capacity) {
  const size_t rows = (size_t)B * Hq * c->cfg.max_tree * cc_splits(c, B, Hkv, Hq / Hkv, page_size, seq_capacity);
  return rows * (D + 2) * sizeof(float);
}

template <typename T, int D>
cast_status launch_cc(cast_ctx* c, AttnParams& p, cudaStream_t s) {
  const int nrowblk = (p.Ncap * p.G + kRB - 1) / kRB;
  const int nsplit = cc_splits(c, p.B, p.Hkv, p.G, p.page_size, p.seq_capacity);
  p.nsplit = nsplit;
  const size_t rows = (size_t)p.B * p.Hq * p.Ncap * nsplit;
  // compute calls never allocate: the workspace comes from cast_reserve_attention
  if (rows * (D + 2) * sizeof(float) > c->attn_ws_bytes) return CAST_ERR_CAPACITY;
  p.part_o = reinterpret_cast<float*>(c->attn_ws);
  p.part_ml = p.part_o + rows * D;
  const size_t smem = (size_t)(kRB * (D + 4) + kPT * (D + 4) + kPT * D + kRB * (kPT + 1)) * sizeof(float);
  CAST_CUDA_OK(cudaFuncSetAttribute(tree_attn_cc_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  tree_attn_cc_kernel<T, D><<<dim3(nsplit * nrowblk, p.Hkv, p.B), kThreads, smem, s>>>(p);
  attn_combine_kernel<T, D><<<dim3(p.Ncap, p.Hq, p.B), D, 0, s>>>(p);
  return launch_status();
}

}  // namespace

extern "C" cast_status cast_set_attention_early_reads(cast_ctx* c, int promise) {
  if (!c) return CAST_ERR_INVALID_ARG;
  c->attn_early = promise ? 1 : 0;
  c->wl_valid = 0;
  return CAST_OK;
}

extern "C" cast_status cast_reserve_attention(cast_ctx* c, cast_dtype dtype, int B, int Hq, int Hkv, int D, int page_size,
                                              int seq_capacity) {
  if (!c || B < 1 || Hq < 1 || Hkv < 1 || page_size < 0 || seq_capacity < 1) return CAST_ERR_INVALID_ARG;
  if (dtype != CAST_F32 && dtype != CAST_BF16) return CAST_ERR_DTYPE;
  if (B > c->cfg.max_batch) return CAST_ERR_CAPACITY;
  if (Hq % Hkv != 0 || (D != 64 && D != 128)) return CAST_ERR_SHAPE;
  // a bf16 call takes the tensor-core path when shape and pointer alignment allow and the CUDA-core path
  // otherwise: both workspaces are sized, so the choice at call time never needs memory
  if (dtype == CAST_BF16) {
    const cast_status st = tree_attention_tc_reserve(c, tree_attention_tc_workspace(c, B, Hq, Hkv, D, page_size, seq_capacity));
    if (st != CAST_OK) return st;
  }
  const size_t need = cc_workspace(c, B, Hq, Hkv, D, page_size, seq_capacity);
  if (need > c->attn_ws_bytes) {
    CAST_CUDA_OK(cudaDeviceSynchronize());
    if (c->attn_ws) cudaFree(c->attn_ws);
    c->attn_ws = nullptr;
    c->attn_ws_bytes = 0;
    CAST_CUDA_OK(cudaMalloc(&c->attn_ws, need));
    c->attn_ws_bytes = need;
  }
  return CAST_OK;
}

extern "C" cast_status cast_tree_attention_rows(cast_ctx* c, const void* q, const void* k_cache, const void* v_cache,
                                                cast_dtype dtype, int B, int Hq, int Hkv, int D, int page_size,
                                                const int32_t* page_table, int seq_capacity, int num_pages,
                                                const int32_t* kv_len, const uint32_t* anc_mask, const int32_t* n_tree,
                                                const int32_t* first_row, float scale, void* out, void* stream) {
  if (!c || !q || !k_cache || !v_cache || !kv_len || !anc_mask || !n_tree || !out || B < 1 || Hq < 1 || Hkv < 1 ||
      page_size < 0 || seq_capacity < 1 || (page_size > 0 && (!page_table || num_pages < 1)))
    return CAST_ERR_INVALID_ARG;
  if (dtype != CAST_F32 && dtype != CAST_BF16) return CAST_ERR_DTYPE;
  if (B > c->cfg.max_batch) return CAST_ERR_CAPACITY;
  if (Hq % Hkv != 0 || (D != 64 && D != 128)) return CAST_ERR_SHAPE;
  if (((uintptr_t)q | (uintptr_t)k_cache | (uintptr_t)v_cache | (uintptr_t)out) & 15) return CAST_ERR_SHAPE;
  if (scale == 0.f) scale = 1.0f / sqrtf((float)D);
  cudaStream_t s = (cudaStream_t)stream;
  const int fresh = c->tree_inputs_fresh;
  c->tree_inputs_fresh = 0;  // whatever is launched below waits for its predecessor before it releases its own dependents
  if (dtype == CAST_BF16) {
    cast_status st = CAST_OK;
    c->tree_inputs_fresh = fresh;
    const bool taken = tree_attention_tc_launch(c, q, k_cache, v_cache, B, Hq, Hkv, D, page_size, page_table, seq_capacity,
                                                num_pages, kv_len, anc_mask, n_tree, first_row, scale, out, s, &st);
    c->tree_inputs_fresh = 0;
    if (taken) return st;
  }
  AttnParams p;
  p.q = q; p.k = k_cache; p.v = v_cache; p.out = out;
  p.B = B; p.Ncap = c->cfg.max_tree; p.Hq = Hq; p.Hkv = Hkv; p.G = Hq / Hkv;
  p.page_size = page_size; p.seq_capacity = seq_capacity; p.num_pages = num_pages; p.words = c->words;
  p.nsplit = 1;
  p.page_table = page_table; p.kv_len = kv_len; p.n_tree = n_tree; p.first_row = first_row; p.anc = anc_mask;
  p.scale = scale; p.part_o = nullptr; p.part_ml = nullptr; p.st = c->state;
  if (dtype == CAST_F32) return D == 64 ? launch_cc<float, 64>(c, p, s) : launch_cc<float, 128>(c, p, s);
  return D == 64 ? launch_cc<__nv_bfloat16, 64>(c, p, s) : launch_cc<__nv_bfloat16, 128>(c, p, s);
}

extern "C" cast_status cast_tree_attention(cast_ctx* c, const void* q, const void* k_cache, const void* v_cache,
                                           cast_dtype dtype, int B, int Hq, int Hkv, int D, int page_size,
                                           const int32_t* page_table, int seq_capacity, int num_pages,
                                           const int32_t* kv_len, const uint32_t* anc_mask, const int32_t* n_tree,
                                           float scale, void* out, void* stream) {
  return cast_tree_attention_rows(c, q, k_cache, v_cache, dtype, B, Hq, Hkv, D, page_size, page_table, seq_capacity,
                                  num_pages, kv_len, anc_mask, n_tree, nullptr, scale, out, stream);
}
