// Tensor-core path of cast_tree_attention for bf16, head_dim 128 (sm_100a: tcgen05 + TMEM + TMA).
//
// One CTA owns (sequence b, kv-head, block of 128 query rows, KV split). A query row is a
// (tree token, head of the GQA group) pair, so every K/V tile is fetched once for all tree
// tokens and all heads of the group. Tiles are 64 positions. Roles:
//   control warp : TMA loads of K and V (128B-swizzled, two 64-column halves each) into a 4-stage
//                  ring; S = Q K^T by tcgen05.mma (M=128 rows, N=64 positions, K=128) into one of
//                  two TMEM buffers; once the softmax warps have written P, O += P V (V is the
//                  MN-major B operand: used exactly as it lies in the cache, no transpose).
//                  QK^T of tile i+1 is issued before P of tile i is awaited, so the tensor pipe
//                  works on the next scores while the softmax of the current tile runs.
//   8 softmax warps: thread (row, column half) reads its 32 scores with tcgen05.ld, applies the
//                  prefix/ancestor mask (only tiles that reach past the prefix need one), keeps a
//                  lazily updated row maximum (O in TMEM is rescaled only when the maximum grows
//                  by more than 2^8), writes P as bf16 into one of two swizzled smem buffers.
// The number of KV splits is decided on the device from the actual tree sizes and prefix
// lengths (the host only fixes its upper bound), so the grid fills the machine whatever N the
// cost model picked. All mbarrier waits are bounded: on expiry the CTA records
// CAST_ERR_TIMEOUT, drains its copies, frees its TMEM and returns.
#include <cuda.h>
#include <math.h>

#include "cast_internal.h"

#ifdef CAST_PHASE_CLOCKS
__device__ long long g_attn_clock[256];
extern "C" __attribute__((visibility("default"))) int cast_debug_read_attn_clocks(long long* out) {
  return (int)cudaMemcpyFromSymbol(out, g_attn_clock, sizeof(long long) * 256);
}
#define TC_STAMP(role, it, k) do { if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && (it) >= 4 && (it) < 8 && \
    (threadIdx.x == ((role) ? 288 : 0))) g_attn_clock[(role) * 128 + ((it) - 4) * 16 + (k)] = clock64(); } while (0)
#define TC_MARK(k) do { if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) g_attn_clock[240 + (k)] = clock64(); } while (0)
#else
#define TC_STAMP(role, it, k) do {} while (0)
#define TC_MARK(k) do {} while (0)
#endif

namespace cast {

namespace {

constexpr int kBM = 128;          // query rows per CTA (UMMA M)
constexpr int kBN = 64;           // positions per tile
constexpr int kHD = 128;          // head dim
constexpr int kStages = 4;        // K/V ring
constexpr int kSoftmaxThreads = 256;
constexpr int kThreadsTC = kSoftmaxThreads + 64;  // + TMA producer warp + MMA issuer warp
constexpr int kRegionQ = kBM * 128;                // [128 rows][64] bf16, 128B rows: 16 KB
constexpr int kRegionKV = kBN * 128;               // [64 positions][64] bf16: 8 KB
constexpr int kSmemQ = 0;                          // 2 regions (d 0-63, d 64-127)
constexpr int kSmemP = 2 * kRegionQ;               // 2 buffers of one region [128 rows][64 positions]
constexpr int kSmemKV = 4 * kRegionQ;              // stage s: K (2 regions) then V (2 regions)
constexpr int kStageBytes = 4 * kRegionKV;         // 32 KB
constexpr int kSmemBytes = kSmemKV + kStages * kStageBytes;  // 192 KB
constexpr int kTmemCols = 256;                     // S0: [0,64), S1: [64,128), O: [128,256)
constexpr float kRescaleThreshold = 8.0f;          // log2 units
constexpr long long kWaitCycles = 4000000000ll;    // about two seconds
constexpr int kMaxSplit = 16;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  int B, Ncap, Hq, Hkv, G, page_size, seq_capacity, num_pages, words, nsplit_max, num_sms;
  const int32_t* page_table;
  const int32_t* kv_len;
  const int32_t* n_tree;
  const uint32_t* anc;
  float scale_log2;
  float* part_o;
  float* part_ml;
  DevState* st;
};

// ---- PTX wrappers -----------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the barrier did not complete within kWaitCycles. Every thread that waits
// on the same phase gets the same answer, so the roles give up together.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  if (mbar_test(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_test(bar, parity)) {
    if (clock64() - t0 > kWaitCycles) return false;
  }
  return true;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_3d(const CUtensorMap* map, void* dst, uint64_t* bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(const CUtensorMap* map, void* dst, uint64_t* bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulation.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void softmax_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kSoftmaxThreads) : "memory"); }

// Byte offset of 16-byte chunk `c` (0..7) of row `r` inside a 128B-swizzled [rows][64 bf16] region.
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

// KV splits actually used, from the tree sizes and prefix lengths on the device: enough CTAs for
// about four waves, at least eight tiles each where the sequences are long enough, and never fewer
// CTAs than SMs when the work allows. Every warp computes the same value.
__device__ __forceinline__ int effective_splits(const TcParams& p) {
  const int lane = threadIdx.x & 31;
  const int max_pos = p.page_size == 0 ? p.seq_capacity : p.seq_capacity * p.page_size;
  int active = 0, tiles = 0;
  for (int b = lane; b < p.B; b += 32) {
    int N = p.n_tree[b];
    N = N < 0 ? 0 : (N > p.Ncap ? p.Ncap : N);
    int L = p.kv_len[b];
    L = L < 0 ? 0 : L;
    int total = L + N;
    total = total > max_pos ? max_pos : total;
    const int nrb = (N * p.G + kBM - 1) / kBM;
    active += p.Hkv * nrb;
    tiles += p.Hkv * nrb * ((total + kBN - 1) / kBN);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    active += __shfl_xor_sync(0xffffffffu, active, o);
    tiles += __shfl_xor_sync(0xffffffffu, tiles, o);
  }
  if (active == 0) return 1;
  const int per = tiles / active;  // mean tiles per (sequence, kv-head, row block)
  int want = active * per / 8;
  want = want > 4 * p.num_sms ? 4 * p.num_sms : want;
  want = want < p.num_sms ? p.num_sms : want;
  int ns = (want + active - 1) / active;
  ns = ns > p.nsplit_max ? p.nsplit_max : ns;
  ns = ns > per ? per : ns;
  return ns < 1 ? 1 : ns;
}

__global__ void __launch_bounds__(kThreadsTC, 1)
tree_attn_tc_kernel(const TcParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kStages], bar_free[kStages], bar_s[2], bar_p[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ float xch[2][kBM * 2];
  __shared__ uint32_t anc_s[kBM][CAST_MAX_TREE / 32];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  TC_MARK(0);
  const int nsplit = effective_splits(p);
  TC_MARK(1);
  const int split = blockIdx.x % p.nsplit_max, rb = blockIdx.x / p.nsplit_max;
  if (split >= nsplit) return;
  const int kvh = blockIdx.y, b = blockIdx.z;
  int N = p.n_tree[b];
  N = N < 0 ? 0 : (N > p.Ncap ? p.Ncap : N);
  int L = p.kv_len[b];
  if (L < 0) L = 0;
  const int G = p.G, rows_total = N * G, row0 = rb * kBM;
  if (row0 >= rows_total) return;
  const int max_pos = p.page_size == 0 ? p.seq_capacity : p.seq_capacity * p.page_size;
  int total = L + N;
  if (total > max_pos) {
    if (tid == 0) report(p.st, CAST_ERR_BAD_PAGE, b);
    total = max_pos;
  }
  const int ntiles = (total + kBN - 1) / kBN;
  const int t0 = (int)((long long)split * ntiles / nsplit), t1 = (int)((long long)(split + 1) * ntiles / nsplit);
  const int ntile = t1 - t0;
  const int half = (warp >> 2) & 1, quarter = warp & 3, r = quarter * 32 + lane;  // softmax-role coordinates
  const int row = row0 + r;
  const bool row_ok = warp < 8 && row < rows_total;
  const int t_tok = row_ok ? row / G : 0, h_q = kvh * G + (row_ok ? row % G : 0);
  const size_t pr = (((size_t)b * p.Hq + h_q) * p.Ncap + t_tok) * p.nsplit_max + split;
  if (ntile <= 0) {  // nothing to attend to in this split: an empty partial
    if (row_ok && half == 0) {
      p.part_ml[pr * 2] = -INFINITY;
      p.part_ml[pr * 2 + 1] = 0.f;
    }
    return;
  }
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);

  // tile j of this CTA -> ring stage j % kStages (producer warp only; all 32 lanes call it)
  auto issue_load = [&](int j) -> bool {
    const int stage = j % kStages;
    unsigned char* kdst = smem + kSmemKV + stage * kStageBytes;
    unsigned char* vdst = kdst + 2 * kRegionKV;
    const int pos0 = (t0 + j) * kBN;
    const int ps = p.page_size;
    int npages = 0, page = 0;
    if (ps != 0) {  // page ids are fetched before the stage is awaited: their latency hides behind the wait
      const int ppt = kBN / ps;
      npages = (total - pos0 + ps - 1) / ps;
      npages = npages > ppt ? ppt : npages;
      if (lane < npages * 4) {
        page = p.page_table[(size_t)b * p.seq_capacity + pos0 / ps + (lane >> 2)];
        if (page < 0 || page >= p.num_pages) {
          report(p.st, CAST_ERR_BAD_PAGE, b);
          page = 0;
        }
      }
    }
    if (j >= kStages) {
      const bool w = mbar_wait(&bar_free[stage], ((j / kStages) - 1) & 1);
      if (!__all_sync(0xffffffffu, w)) return false;
    }
    if (ps == 0) {
      if (lane == 0) mbar_expect_tx(&bar_full[stage], kStageBytes);
      __syncwarp();
      if (lane < 4) {
        const int hsel = lane & 1;
        tma_load_3d(lane < 2 ? &map_k : &map_v, (lane < 2 ? kdst : vdst) + hsel * kRegionKV, &bar_full[stage], hsel * 64,
                    kvh, b * p.seq_capacity + pos0);
      }
    } else {  // at most 8 pages per tile (page size >= 8): one (page, tensor, half) per lane
      if (lane == 0) mbar_expect_tx(&bar_full[stage], (uint32_t)npages * ps * 128 * 4);
      __syncwarp();
      if (lane < npages * 4) {
        const int slot = lane >> 2, which = lane & 3, hsel = which & 1;
        tma_load_4d(which < 2 ? &map_k : &map_v, (which < 2 ? kdst : vdst) + hsel * kRegionKV + slot * ps * 128,
                    &bar_full[stage], hsel * 64, kvh, 0, page);
      }
    }
    __syncwarp();
    return true;
  };

  int armed = 0;
  bool prod_ok = true;
  if (warp == 8) {
    if (lane == 0) {
      for (int s = 0; s < kStages; ++s) {
        mbar_init(&bar_full[s], 1);
        mbar_init(&bar_free[s], 1);
      }
      for (int s = 0; s < 2; ++s) {
        mbar_init(&bar_s[s], 1);
        mbar_init(&bar_p[s], kSoftmaxThreads);
      }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_proxy_async();
    }
    __syncwarp();
    for (int j = 0; j < kStages && j < ntile; ++j) {  // the ring fills while the other warps stage Q
      prod_ok = issue_load(j);
      armed = j + 1;
    }
  } else if (warp < 8) {
    if (warp == 0) {  // TMEM: two S buffers and O
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)),
                   "n"(kTmemCols));
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    // Q rows -> swizzled shared memory (rows past the tree are zero); ancestor masks
    const __nv_bfloat16* qrow = p.q + (((size_t)b * p.Ncap + t_tok) * p.Hq + h_q) * kHD + half * 64;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (row_ok) v = *reinterpret_cast<const uint4*>(qrow + c * 8);
      *reinterpret_cast<uint4*>(smem + kSmemQ + half * kRegionQ + swz(r, c)) = v;
    }
    if (half == 0) {
      for (int w = 0; w < CAST_MAX_TREE / 32; ++w)
        anc_s[r][w] = (row_ok && w < p.words) ? p.anc[((size_t)b * p.Ncap + t_tok) * p.words + w] : 0u;
    }
    fence_proxy_async();
  }
  TC_MARK(2);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  TC_MARK(3);
  const uint32_t tmem_base = tmem_base_s;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + 2 * kBN;

  if (warp == 8) {
    // =========================== TMA producer ===========================
    bool ok = prod_ok;
    for (int j = armed; ok && j < ntile; ++j) {
      ok = issue_load(j);
      if (ok) armed = j + 1;
    }
    if (!ok) {  // drain: copies in flight must land before the CTA's shared memory is released
      if (lane == 0) report(p.st, CAST_ERR_TIMEOUT, b);
      for (int j = (armed > kStages ? armed - kStages : 0); j < armed; ++j) {
        const long long tw = clock64();
        while (!mbar_test(&bar_full[j % kStages], (j / kStages) & 1) && clock64() - tw < kWaitCycles) {}
      }
    }
  } else if (warp == 9) {
    // =========================== MMA issuer ===========================
    const uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
    const uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(kHD >> 3) << 17) |
                              ((uint32_t)(kBM >> 4) << 24);  // B operand (V) is MN-major, N = head dim
    // descriptors differ only in the start-address field (16-byte units), so they are built once
    const uint64_t dq = umma_desc(smem_u32(smem + kSmemQ), 16, 1024);
    const uint64_t dk = umma_desc(smem_u32(smem + kSmemKV), 16, 1024);
    const uint64_t dv = umma_desc(smem_u32(smem + kSmemKV + 2 * kRegionKV), kRegionKV, 1024);
    const uint64_t dp = umma_desc(smem_u32(smem + kSmemP), 16, 1024);
    auto mma_qk = [&](int stage, int buf) {  // S[buf] = Q K^T
      if (lane == 0) {
        const uint64_t dks = dk + (uint64_t)(stage * (kStageBytes >> 4));
#pragma unroll
        for (int ks = 0; ks < kHD / 16; ++ks)
          umma_bf16(tmem_s + buf * kBN, dq + (uint64_t)((ks >> 2) * (kRegionQ >> 4) + (ks & 3) * 2),
                    dks + (uint64_t)((ks >> 2) * (kRegionKV >> 4) + (ks & 3) * 2), idesc_qk, ks > 0);
        umma_commit(&bar_s[buf]);
      }
      __syncwarp();
    };
    auto mma_pv = [&](int stage, int buf, bool first) {  // O (+)= P[buf] V
      if (lane == 0) {
        const uint64_t dvs = dv + (uint64_t)(stage * (kStageBytes >> 4));
        const uint64_t dpb = dp + (uint64_t)(buf * (kRegionQ >> 4));
#pragma unroll
        for (int ks = 0; ks < kBN / 16; ++ks)
          umma_bf16(tmem_o, dpb + (uint64_t)(ks * 2), dvs + (uint64_t)(ks * (2048 >> 4)), idesc_pv,
                    (!first || ks > 0) ? 1u : 0u);
        umma_commit(&bar_free[stage]);
      }
      __syncwarp();
    };
    auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
      const bool w = mbar_wait(bar, parity);
      return __all_sync(0xffffffffu, w);
    };
    bool ok = wait_all(&bar_full[0], 0);
    if (ok) {
      tc_fence_after();
      mma_qk(0, 0);
    }
    for (int it = 0; ok && it < ntile; ++it) {
      TC_STAMP(1, it, 0);
      if (it + 1 < ntile) {  // next scores first: they are computed while the softmax of tile `it` runs
        ok = wait_all(&bar_full[(it + 1) % kStages], ((it + 1) / kStages) & 1);
        if (!ok) break;
        TC_STAMP(1, it, 1);
        tc_fence_after();
        mma_qk((it + 1) % kStages, (it + 1) & 1);
        TC_STAMP(1, it, 2);
      }
      ok = wait_all(&bar_p[it & 1], (it >> 1) & 1);
      if (!ok) break;
      TC_STAMP(1, it, 3);
      tc_fence_after();
      mma_pv(it % kStages, it & 1, it == 0);
      TC_STAMP(1, it, 4);
    }
    if (!ok && lane == 0) report(p.st, CAST_ERR_TIMEOUT, b);
  } else {
    // =========================== softmax warps ===========================
    // After a wait has expired a thread keeps visiting the barriers (so nobody blocks on it) but
    // touches neither TMEM nor the operand buffers. A warp whose 32 rows all lie past the tree
    // only keeps the barriers in step: its P rows feed output rows nobody reads.
    const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
    const bool warp_live = row0 + quarter * 32 < rows_total;
    const float sc = p.scale_log2;
    float m_used = -INFINITY, l_run = 0.f;  // m_used: running reference maximum in raw score units
    bool ok = true;
    for (int it = 0; it < ntile; ++it) {
      const int buf = it & 1, stage = it % kStages;
      const int pos0 = (t0 + it) * kBN;
      uint32_t sr[32];
      float mx = -INFINITY;
      TC_STAMP(0, it, 0);
      if (warp_live) {
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bar_s[buf], (it >> 1) & 1));
        TC_STAMP(0, it, 1);
        if (ok) {
          tc_fence_after();
          tmem_ld32(tmem_s + buf * kBN + lane_sel + half * 32, sr);
          tmem_wait_ld();
          TC_STAMP(0, it, 2);
          const int cbase = pos0 + half * 32;
          if (cbase + 32 > L) {  // this thread's 32 columns reach past the prefix: ancestor mask
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int pos = cbase + c;
              bool v = pos < L;
              if (!v && pos < total) {
                const int j = pos - L;
                v = (anc_s[r][j >> 5] >> (j & 31)) & 1u;
              }
              if (!v) sr[c] = 0xff800000u;  // -inf
            }
          }
          float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
          for (int c = 0; c < 32; c += 4) {
            m0 = fmaxf(m0, __uint_as_float(sr[c]));
            m1 = fmaxf(m1, __uint_as_float(sr[c + 1]));
            m2 = fmaxf(m2, __uint_as_float(sr[c + 2]));
            m3 = fmaxf(m3, __uint_as_float(sr[c + 3]));
          }
          mx = row_ok ? fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) : -INFINITY;
        }
      }
      TC_STAMP(0, it, 3);
      xch[buf][half * kBM + r] = mx;
      softmax_bar();
      mx = fmaxf(mx, xch[buf][(half ^ 1) * kBM + r]);
      TC_STAMP(0, it, 4);
      if (warp_live && ok) {
        // lazy maximum: move the reference only when the row maximum outgrows it by 2^8
        float alpha = 1.f;
        const bool grow = (mx - m_used) * sc > kRescaleThreshold || (m_used == -INFINITY && mx > -INFINITY);
        if (grow) {
          alpha = fast_exp2((m_used - mx) * sc);  // 0 when m_used = -inf
          m_used = mx;
          l_run *= alpha;
        }
        if (it > 0 && __any_sync(0xffffffffu, grow)) {  // rescale this thread's 64 columns of O
          ok = __all_sync(0xffffffffu, mbar_wait(&bar_free[(it - 1) % kStages], ((it - 1) / kStages) & 1));
          if (ok) {
            tc_fence_after();
            uint32_t orr[32];
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
              const uint32_t ta = tmem_o + lane_sel + half * 64 + hh * 32;
              tmem_ld32(ta, orr);
              tmem_wait_ld();
#pragma unroll
              for (int c = 0; c < 32; ++c) orr[c] = __float_as_uint(__uint_as_float(orr[c]) * alpha);
              tmem_st32(ta, orr);
            }
            tmem_wait_st();
          }
        }
        TC_STAMP(0, it, 5);
        // the P buffer was last read by the P V product of tile it-2
        if (ok && it >= 2)
          ok = __all_sync(0xffffffffu, mbar_wait(&bar_free[(it - 2) % kStages], ((it - 2) / kStages) & 1));
        TC_STAMP(0, it, 6);
        if (ok) {
          // P = 2^((s - m) * scale) as bf16 into the swizzled A-operand buffer; row sum in fp32
          const bool live = m_used > -INFINITY;
          const float neg_ms = live ? -m_used * sc : 0.f;
          float l0 = 0.f, l1 = 0.f;
          unsigned char* prow = smem + kSmemP + buf * kRegionQ;
#pragma unroll
          for (int c8 = 0; c8 < 4; ++c8) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              float p0 = fast_exp2(fmaf(__uint_as_float(sr[c8 * 8 + 2 * e]), sc, neg_ms));
              float p1 = fast_exp2(fmaf(__uint_as_float(sr[c8 * 8 + 2 * e + 1]), sc, neg_ms));
              if (!live) p0 = p1 = 0.f;
              l0 += p0;
              l1 += p1;
              const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
              pk[e] = *reinterpret_cast<const uint32_t*>(&pb);
            }
            *reinterpret_cast<uint4*>(prow + swz(r, half * 4 + c8)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
          l_run += l0 + l1;
        }
      }
      // V rows past the end of the sequence may hold anything (0 * NaN would poison O): zero them
      if (ok && total - pos0 < kBN) {
        if (!warp_live) ok = __all_sync(0xffffffffu, mbar_wait(&bar_s[buf], (it >> 1) & 1));  // V has landed by then
        if (ok) {
          const int valid = total - pos0;
          unsigned char* vbase = smem + kSmemKV + stage * kStageBytes + 2 * kRegionKV;
          for (int i = tid; i < (kBN - valid) * 16; i += kSoftmaxThreads) {
            const int rr = valid + (i >> 4), reg = (i >> 3) & 1, c = i & 7;
            *reinterpret_cast<uint4*>(vbase + reg * kRegionKV + rr * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      }
      TC_STAMP(0, it, 7);
      fence_proxy_async();
      tc_fence_before();
      mbar_arrive(&bar_p[buf]);
      TC_STAMP(0, it, 9);
    }
    // epilogue: wait for the last P V, read O, normalise or emit the partial
    TC_MARK(4);
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bar_free[(ntile - 1) % kStages], ((ntile - 1) / kStages) & 1));
    TC_MARK(5);
    xch[0][half * kBM + r] = l_run;
    softmax_bar();
    if (ok && warp_live) {
      tc_fence_after();
      const float l_tot = l_run + xch[0][(half ^ 1) * kBM + r];
      uint32_t orr[64];
      tmem_ld32(tmem_o + lane_sel + half * 64, orr);
      tmem_ld32(tmem_o + lane_sel + half * 64 + 32, orr + 32);
      tmem_wait_ld();
      if (row_ok) {
        if (nsplit == 1) {
          const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
          __nv_bfloat16* orow = p.out + (((size_t)b * p.Ncap + t_tok) * p.Hq + h_q) * kHD + half * 64;
#pragma unroll
          for (int c8 = 0; c8 < 8; ++c8) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const __nv_bfloat162 ob = __floats2bfloat162_rn(__uint_as_float(orr[c8 * 8 + 2 * e]) * inv,
                                                              __uint_as_float(orr[c8 * 8 + 2 * e + 1]) * inv);
              pk[e] = *reinterpret_cast<const uint32_t*>(&ob);
            }
            *reinterpret_cast<uint4*>(orow + c8 * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        } else {
          float* po = p.part_o + pr * kHD + half * 64;
#pragma unroll
          for (int c4 = 0; c4 < 16; ++c4)
            *reinterpret_cast<float4*>(po + c4 * 4) =
                make_float4(__uint_as_float(orr[c4 * 4]), __uint_as_float(orr[c4 * 4 + 1]),
                            __uint_as_float(orr[c4 * 4 + 2]), __uint_as_float(orr[c4 * 4 + 3]));
          if (half == 0) {
            p.part_ml[pr * 2] = m_used * sc * 0.69314718055994531f;  // natural-log units
            p.part_ml[pr * 2 + 1] = l_tot;
          }
        }
      }
    }
  }
  TC_MARK(6);
  tc_fence_before();
  __syncthreads();
  TC_MARK(7);
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols));
  }
}

// Rows >= n_tree of `out` are zeros; split partials are merged (natural-log maxima).
__global__ void __launch_bounds__(kHD) tc_combine_kernel(const TcParams p) {
  const int t = blockIdx.x, h = blockIdx.y, b = blockIdx.z, d = threadIdx.x;
  __nv_bfloat16* out = p.out + (((size_t)b * p.Ncap + t) * p.Hq + h) * kHD;
  int N = p.n_tree[b];
  N = N > p.Ncap ? p.Ncap : N;
  if (t >= N) {
    out[d] = __float2bfloat16_rn(0.f);
    return;
  }
  const int nsplit = effective_splits(p);
  if (nsplit == 1) return;  // written by the attention kernel itself
  const size_t pr = (((size_t)b * p.Hq + h) * p.Ncap + t) * p.nsplit_max;
  float M = -INFINITY;
  for (int s = 0; s < nsplit; ++s) M = fmaxf(M, p.part_ml[(pr + s) * 2]);
  float l = 0.f, acc = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    const float ms = p.part_ml[(pr + s) * 2];
    if (ms > -INFINITY) {
      const float w = expf(ms - M);
      l += p.part_ml[(pr + s) * 2 + 1] * w;
      acc += p.part_o[(pr + s) * kHD + d] * w;
    }
  }
  out[d] = __float2bfloat16_rn(l > 0.f ? acc / l : 0.f);
}

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

bool make_kv_map(CUtensorMap* map, const void* base, int B, int Hkv, int page_size, int seq_capacity, int num_pages) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  const cuuint64_t row_bytes = (cuuint64_t)Hkv * kHD * 2;
  if (page_size == 0) {
    const cuuint64_t dims[3] = {kHD, (cuuint64_t)Hkv, (cuuint64_t)B * seq_capacity};
    const cuuint64_t strides[2] = {kHD * 2, row_bytes};
    const cuuint32_t box[3] = {64, 1, kBN};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  }
  const cuuint64_t dims[4] = {kHD, (cuuint64_t)Hkv, (cuuint64_t)page_size, (cuuint64_t)num_pages};
  const cuuint64_t strides[3] = {kHD * 2, row_bytes, row_bytes * page_size};
  const cuuint32_t box[4] = {64, 1, (cuuint32_t)page_size, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool tree_attention_tc_launch(cast_ctx* c, const void* q, const void* k, const void* v, int B, int Hq, int Hkv, int D,
                              int page_size, const int32_t* page_table, int seq_capacity, int num_pages,
                              const int32_t* kv_len, const uint32_t* anc, const int32_t* n_tree, float scale, void* out,
                              cudaStream_t stream, cast_status* status) {
  if (D != kHD || !(scale > 0.f)) return false;
  if (page_size != 0 && (page_size < 8 || page_size > kBN || (kBN % page_size) != 0 || (page_size % 8) != 0))
    return false;
  if ((((uintptr_t)k | (uintptr_t)v) & 127) != 0) return false;
  CUtensorMap map_k, map_v;
  if (!make_kv_map(&map_k, k, B, Hkv, page_size, seq_capacity, num_pages) ||
      !make_kv_map(&map_v, v, B, Hkv, page_size, seq_capacity, num_pages))
    return false;
  const int G = Hq / Hkv, Ncap = c->cfg.max_tree;
  const int nrb = (Ncap * G + kBM - 1) / kBM;
  const int max_pos = page_size == 0 ? seq_capacity : seq_capacity * page_size;
  const int max_tiles = (max_pos + kBN - 1) / kBN;
  // upper bound of the KV splits; the kernel picks the actual number from the device-side sizes
  int nsplit_max = (4 * c->num_sms + B * Hkv - 1) / (B * Hkv);
  if (nsplit_max > max_tiles) nsplit_max = max_tiles;
  if (nsplit_max > kMaxSplit) nsplit_max = kMaxSplit;
  if (nsplit_max < 1) nsplit_max = 1;
  TcParams p;
  p.q = (const __nv_bfloat16*)q; p.out = (__nv_bfloat16*)out;
  p.B = B; p.Ncap = Ncap; p.Hq = Hq; p.Hkv = Hkv; p.G = G; p.page_size = page_size; p.seq_capacity = seq_capacity;
  p.num_pages = num_pages; p.words = c->words; p.nsplit_max = nsplit_max; p.num_sms = c->num_sms;
  p.page_table = page_table; p.kv_len = kv_len; p.n_tree = n_tree; p.anc = anc;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.part_o = nullptr; p.part_ml = nullptr; p.st = c->state;
  *status = CAST_OK;
  if (nsplit_max > 1) {
    const size_t rows = (size_t)B * Hq * Ncap * nsplit_max;
    const size_t need = rows * (kHD + 2) * sizeof(float);
    if (need > c->attn_ws_bytes) {  // grows the workspace (synchronises; not legal during graph capture)
      if (cudaDeviceSynchronize() != cudaSuccess) { *status = CAST_ERR_CUDA; return true; }
      if (c->attn_ws) cudaFree(c->attn_ws);
      c->attn_ws = nullptr;
      c->attn_ws_bytes = 0;
      if (cudaMalloc(&c->attn_ws, need) != cudaSuccess) { *status = CAST_ERR_CUDA; return true; }
      c->attn_ws_bytes = need;
    }
    p.part_o = reinterpret_cast<float*>(c->attn_ws);
    p.part_ml = p.part_o + rows * kHD;
  }
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(tree_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes + 1024) !=
        cudaSuccess) {
      *status = CAST_ERR_CUDA;
      return true;
    }
    attr_done = true;
  }
  tree_attn_tc_kernel<<<dim3(nsplit_max * nrb, Hkv, B), kThreadsTC, kSmemBytes + 1024, stream>>>(p, map_k, map_v);
  tc_combine_kernel<<<dim3(Ncap, Hq, B), kHD, 0, stream>>>(p);
  *status = launch_status();
  return true;
}

}  // namespace cast
