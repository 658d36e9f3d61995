// Tensor-core path of cast_tree_attention for bf16, head_dim 128 (sm_100a: tcgen05 + TMEM + TMA).
//
// One CTA owns (sequence b, kv-head, block of 128 query rows, KV split). A query row is a
// (tree token, head of the GQA group) pair, so every K/V tile is fetched once for all tree
// tokens and all heads of the group. Tiles are 128 positions. Roles (10 warps):
//   TMA producer : K tiles and V tiles (128B-swizzled, two 64-column halves each) into two
//                  2-stage rings; a K stage is released as soon as Q K^T has consumed it, a V
//                  stage after P V, so K runs about two tiles ahead of the tensor pipe.
//   MMA issuer   : S = Q K^T by tcgen05.mma (M=128 rows, N=128 positions, K=128) into one of two
//                  TMEM buffers; once the softmax warps have written P, O += P V (V is the
//                  MN-major B operand: used exactly as it lies in the cache, no transpose).
//                  Q K^T of tile i+1 is issued before P of tile i is awaited, so the tensor pipe
//                  works on the next scores while the softmax of the current tile runs.
//   8 softmax warps: thread (row, column half) reads its 64 scores with tcgen05.ld, applies the
//                  prefix/ancestor mask (only tiles that reach past the prefix need one), keeps a
//                  lazily updated row maximum (O in TMEM is rescaled only when the maximum grows
//                  by more than 2^8), writes P as bf16 into swizzled shared memory.
// The number of KV splits is decided on the device from the actual tree sizes and prefix
// lengths (the host only fixes its upper bound), so the grid fills the machine whatever N the
// cost model picked. Split partials are merged by the last CTA of a row block to finish (an
// atomic ticket; nothing spins). All mbarrier waits are bounded: on expiry the CTA records
// CAST_ERR_TIMEOUT, drains its copies, frees its TMEM and returns.
#include <cuda.h>
#include <math.h>

#include "cast_internal.h"

#ifdef CAST_PHASE_CLOCKS
__device__ long long g_attn_clock[256];
extern "C" __attribute__((visibility("default"))) int cast_debug_read_attn_clocks(long long* out) {
  return (int)cudaMemcpyFromSymbol(out, g_attn_clock, sizeof(long long) * 256);
}
#define TC_STAMP(role, it, k) do { if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && (it) >= 2 && (it) < 6 && \
    (threadIdx.x == ((role) ? 288 : 0))) g_attn_clock[(role) * 128 + ((it) - 2) * 16 + (k)] = clock64(); } while (0)
#define TC_MARK(k) do { if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) g_attn_clock[240 + (k)] = clock64(); } while (0)
__device__ unsigned long long g_cta_log[4 * 16384];
extern "C" __attribute__((visibility("default"))) int cast_debug_read_cta_log(unsigned long long* out) {
  return (int)cudaMemcpyFromSymbol(out, g_cta_log, sizeof(unsigned long long) * 4 * 16384);
}
__device__ __forceinline__ unsigned long long gtimer() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
__device__ __forceinline__ unsigned smid() { unsigned s; asm volatile("mov.u32 %0, %smid;" : "=r"(s)); return s; }
#define TC_CTA_LOG(k, v) do { if (threadIdx.x == 0) { unsigned _id = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z); if (_id < 16384) g_cta_log[_id * 4 + (k)] = (v); } } while (0)
#else
#define TC_CTA_LOG(k, v) do {} while (0)
#define TC_STAMP(role, it, k) do {} while (0)
#define TC_MARK(k) do {} while (0)
#endif

namespace cast {

namespace {

constexpr int kBM = 128;          // query rows per CTA (UMMA M)
constexpr int kBN = 128;          // positions per tile
constexpr int kHD = 128;          // head dim
constexpr int kStages = 2;        // K ring and V ring
constexpr int kSoftmaxThreads = 256;
constexpr int kThreadsTC = kSoftmaxThreads + 64;  // + TMA producer warp + MMA issuer warp
constexpr int kRegion = 128 * 128;                 // [128 rows][64] bf16, 128-byte rows: 16 KB
constexpr int kTile = 2 * kRegion;                 // a [128][128] bf16 operand: 32 KB
constexpr int kSmemQ = 0;
constexpr int kSmemP = kTile;
constexpr int kSmemK = 2 * kTile;                  // kStages tiles
constexpr int kSmemV = kSmemK + kStages * kTile;   // kStages tiles
constexpr int kSmemBytes = kSmemV + kStages * kTile;  // 192 KB
constexpr int kTmemCols = 512;                     // S0: [0,128), S1: [128,256), O: [256,384)
constexpr float kRescaleThreshold = 8.0f;          // log2 units
constexpr long long kWaitCycles = 4000000000ll;    // about two seconds
constexpr int kMaxSplit = 8;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  int B, Ncap, Nmax, Hq, Hkv, G, page_size, seq_capacity, num_pages, words, nsplit_max, num_sms, nrb;
  const int32_t* page_table;
  const int32_t* kv_len;
  const int32_t* n_tree;
  const uint32_t* anc;
  float scale_log2;
  float* part_o;     // [B][Hq][Ncap][nsplit_max][D]
  float* part_ml;    // [B][Hq][Ncap][nsplit_max][2]
  int32_t* ticket;   // [B][Hkv][nrb]
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
// Bounded wait with a warp-uniform result (all 32 lanes must call it): false when the barrier did
// not complete within kWaitCycles.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  bool done = mbar_test(bar, parity);
  if (!done) {
    const long long t0 = clock64();
    while (!(done = mbar_test(bar, parity))) {
      if (clock64() - t0 > kWaitCycles) break;
    }
  }
  return __all_sync(0xffffffffu, done);
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

__device__ __forceinline__ int clampi(int x, int lo, int hi) { return x < lo ? lo : (x > hi ? hi : x); }

// Per-sequence sizes and the number of KV splits actually used, from the tree sizes and prefix
// lengths on the device: enough CTAs for about four waves, at least four tiles each where the
// sequences are long enough, and never fewer CTAs than SMs when the work allows. Every warp
// computes the same values (all 32 lanes must call). *N_b and *L_b receive the sizes of sequence b.
__device__ __forceinline__ int effective_splits(const TcParams& p, int b, int* N_b, int* L_b) {
  const int lane = threadIdx.x & 31;
  const int max_pos = p.page_size == 0 ? p.seq_capacity : p.seq_capacity * p.page_size;
  int active = 0, tiles = 0, Nb = 0, Lb = 0;
  for (int b0 = 0; b0 < p.B; b0 += 32) {
    const int bb = b0 + lane;
    int N = 0, L = 0;
    if (bb < p.B) {
      N = clampi(p.n_tree[bb], 0, p.Nmax);
      L = p.kv_len[bb];
      L = L < 0 ? 0 : L;
    }
    int total = L + N;
    total = total > max_pos ? max_pos : total;
    const int nrb = (N * p.G + kBM - 1) / kBM;
    active += p.Hkv * nrb;
    tiles += p.Hkv * nrb * ((total + kBN - 1) / kBN);
    if (b >= b0 && b < b0 + 32) {
      Nb = __shfl_sync(0xffffffffu, N, b - b0);
      Lb = __shfl_sync(0xffffffffu, L, b - b0);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    active += __shfl_xor_sync(0xffffffffu, active, o);
    tiles += __shfl_xor_sync(0xffffffffu, tiles, o);
  }
  *N_b = Nb;
  *L_b = Lb;
  if (active == 0) return 1;
  const int per = tiles / active;  // mean tiles per (sequence, kv-head, row block)
  int want = active * per / 4;
  want = want > 4 * p.num_sms ? 4 * p.num_sms : want;
  want = want < p.num_sms ? p.num_sms : want;
  int ns = (want + active - 1) / active;
  ns = ns > p.nsplit_max ? p.nsplit_max : ns;
  return ns < 1 ? 1 : ns;
}

__global__ void __launch_bounds__(kThreadsTC, 1)
tree_attn_tc_kernel(const TcParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t bar_fullk[kStages], bar_fullv[kStages], bar_freek[kStages], bar_freev[kStages],
      bar_s[2], bar_p;
  __shared__ uint32_t tmem_base_s;
  __shared__ int last_s;
  __shared__ float xch[2][kBM * 2];
  __shared__ uint32_t anc_s[kBM][CAST_MAX_TREE / 32];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x % p.nsplit_max, rb = blockIdx.x / p.nsplit_max;
  const int kvh = blockIdx.y, b = blockIdx.z;
  TC_MARK(0);
  TC_CTA_LOG(0, gtimer());
  TC_CTA_LOG(1, 0ull);
  TC_CTA_LOG(3, 0ull);
  TC_CTA_LOG(2, (unsigned long long)smid());
  int N, L;
  int nsplit = effective_splits(p, b, &N, &L);
  TC_MARK(1);
  const int G = p.G, rows_total = N * G, row0 = rb * kBM;
  if (tid == 0 && rb == 0 && split == 0 && kvh == 0 && p.n_tree[b] > p.Nmax) report(p.st, CAST_ERR_BAD_TREE, b);
  if (row0 >= rows_total) return;
  const int max_pos = p.page_size == 0 ? p.seq_capacity : p.seq_capacity * p.page_size;
  int total = L + N;
  if (total > max_pos) {
    if (tid == 0) report(p.st, CAST_ERR_BAD_PAGE, b);
    total = max_pos;
  }
  const int ntiles = (total + kBN - 1) / kBN;  // >= 1 because N >= 1 here
  nsplit = nsplit > ntiles ? ntiles : nsplit;  // this sequence's splits: none of them is empty
  if (split >= nsplit) return;
  const int t0 = (int)((long long)split * ntiles / nsplit), t1 = (int)((long long)(split + 1) * ntiles / nsplit);
  const int ntile = t1 - t0;
  const int half = (warp >> 2) & 1, quarter = warp & 3, r = quarter * 32 + lane;  // softmax-role coordinates
  const int row = row0 + r;
  const bool row_ok = warp < 8 && row < rows_total;
  const int t_tok = row_ok ? row / G : 0, h_q = kvh * G + (row_ok ? row % G : 0);
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);

  // ---- producer helpers (warp 8; all 32 lanes call them) ----
  // which = 0: K tile j into the K ring, which = 1: V tile j into the V ring
  auto issue_tile = [&](int j, int which) -> bool {
    const int stage = j % kStages;
    unsigned char* dst = smem + (which ? kSmemV : kSmemK) + stage * kTile;
    uint64_t* full = which ? &bar_fullv[stage] : &bar_fullk[stage];
    const CUtensorMap* map = which ? &map_v : &map_k;
    const int pos0 = (t0 + j) * kBN;
    const int ps = p.page_size;
    int npages = 0, page = 0;
    if (ps != 0) {  // page ids are fetched before the stage is awaited: their latency hides behind the wait
      const int ppt = kBN / ps;
      npages = (total - pos0 + ps - 1) / ps;
      npages = npages > ppt ? ppt : npages;
      if (lane < npages * 2) {
        page = p.page_table[(size_t)b * p.seq_capacity + pos0 / ps + (lane >> 1)];
        if (page < 0 || page >= p.num_pages) {
          report(p.st, CAST_ERR_BAD_PAGE, b);
          page = 0;
        }
      }
    }
    if (j >= kStages && !mbar_wait(which ? &bar_freev[stage] : &bar_freek[stage], ((j / kStages) - 1) & 1)) return false;
    if (ps == 0) {
      if (lane == 0) mbar_expect_tx(full, kTile);
      __syncwarp();
      if (lane < 2) tma_load_3d(map, dst + lane * kRegion, full, lane * 64, kvh, b * p.seq_capacity + pos0);
    } else {  // at most 16 pages per tile (page size >= 8): one (page, column half) per lane
      if (lane == 0) mbar_expect_tx(full, (uint32_t)npages * ps * 128 * 2);
      __syncwarp();
      if (lane < npages * 2) {
        const int slot = lane >> 1, hsel = lane & 1;
        tma_load_4d(map, dst + hsel * kRegion + slot * ps * 128, full, hsel * 64, kvh, 0, page);
      }
    }
    __syncwarp();
    return true;
  };
  // issue order K0 K1 V0 K2 V1 K3 V2 ...: the order in which the stages come free
  auto issue_seq = [&](int i, int* armed_k, int* armed_v) -> bool {  // i-th element of that sequence
    int j, which;
    if (i == 0) { j = 0; which = 0; }
    else if (i & 1) { j = (i + 1) / 2; which = 0; }
    else { j = i / 2 - 1; which = 1; }
    if (j >= ntile) return true;
    if (!issue_tile(j, which)) return false;
    if (which) *armed_v = j + 1; else *armed_k = j + 1;
    return true;
  };

  int armed_k = 0, armed_v = 0;
  bool prod_ok = true;
  if (warp == 8) {
    if (lane == 0) {
      for (int s = 0; s < kStages; ++s) {
        mbar_init(&bar_fullk[s], 1);
        mbar_init(&bar_fullv[s], 1);
        mbar_init(&bar_freek[s], 1);
        mbar_init(&bar_freev[s], 1);
      }
      mbar_init(&bar_s[0], 1);
      mbar_init(&bar_s[1], 1);
      mbar_init(&bar_p, kSoftmaxThreads);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_proxy_async();
    }
    __syncwarp();
    // K0 K1 V0 V1 need no stage wait: the rings fill while the other warps stage Q
    for (int i = 0; i < 5 && prod_ok; ++i) {
      if (i == 3) continue;  // K2 waits for a stage; V1 (element 4) does not
      prod_ok = issue_seq(i, &armed_k, &armed_v);
    }
  } else if (warp < 8) {
    if (warp == 0) {  // TMEM: two S buffers and O
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)),
                   "n"(kTmemCols));
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    // Q rows -> swizzled shared memory (rows past the tree are zero); ancestor masks
    const __nv_bfloat16* qrow = p.q + (((size_t)b * p.Ncap + t_tok) * p.Hq + h_q) * kHD + half * 64;
    uint4 qv[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) qv[c] = row_ok ? *reinterpret_cast<const uint4*>(qrow + c * 8) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(smem + kSmemQ + half * kRegion + swz(r, c)) = qv[c];
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
    if (ok) ok = issue_seq(3, &armed_k, &armed_v);  // K2
    for (int i = 5; ok && i <= 2 * ntile; ++i) ok = issue_seq(i, &armed_k, &armed_v);
    if (!ok) {  // drain: copies in flight must land before the CTA's shared memory is released
      if (lane == 0) report(p.st, CAST_ERR_TIMEOUT, b);
      for (int w = 0; w < 2; ++w) {
        const int armed = w ? armed_v : armed_k;
        for (int j = (armed > kStages ? armed - kStages : 0); j < armed; ++j) {
          const long long tw = clock64();
          while (!mbar_test(w ? &bar_fullv[j % kStages] : &bar_fullk[j % kStages], (j / kStages) & 1) &&
                 clock64() - tw < kWaitCycles) {}
        }
      }
    }
  } else if (warp == 9) {
    // =========================== MMA issuer ===========================
    const uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
    const uint32_t idesc_pv = idesc_qk | (1u << 16);  // B operand (V) is MN-major; N = head dim = 128 as well
    // descriptors differ only in the start-address field (16-byte units), so they are built once
    const uint64_t dq = umma_desc(smem_u32(smem + kSmemQ), 16, 1024);
    const uint64_t dk = umma_desc(smem_u32(smem + kSmemK), 16, 1024);
    const uint64_t dv = umma_desc(smem_u32(smem + kSmemV), kRegion, 1024);
    const uint64_t dp = umma_desc(smem_u32(smem + kSmemP), 16, 1024);
    auto mma_qk = [&](int stage, int buf) {  // S[buf] = Q K^T; releases the K stage
      if (lane == 0) {
        const uint64_t dks = dk + (uint64_t)(stage * (kTile >> 4));
#pragma unroll
        for (int ks = 0; ks < kHD / 16; ++ks) {
          const uint64_t off = (uint64_t)((ks >> 2) * (kRegion >> 4) + (ks & 3) * 2);
          umma_bf16(tmem_s + buf * kBN, dq + off, dks + off, idesc_qk, ks > 0);
        }
        umma_commit(&bar_s[buf]);
        umma_commit(&bar_freek[stage]);
      }
      __syncwarp();
    };
    auto mma_pv = [&](int stage, bool first) {  // O (+)= P V; releases the V stage (and P)
      if (lane == 0) {
        const uint64_t dvs = dv + (uint64_t)(stage * (kTile >> 4));
#pragma unroll
        for (int ks = 0; ks < kBN / 16; ++ks)
          umma_bf16(tmem_o, dp + (uint64_t)((ks >> 2) * (kRegion >> 4) + (ks & 3) * 2), dvs + (uint64_t)(ks * (2048 >> 4)),
                    idesc_pv, (!first || ks > 0) ? 1u : 0u);
        umma_commit(&bar_freev[stage]);
      }
      __syncwarp();
    };
    bool ok = mbar_wait(&bar_fullk[0], 0);
    if (ok) {
      tc_fence_after();
      mma_qk(0, 0);
    }
    for (int it = 0; ok && it < ntile; ++it) {
      TC_STAMP(1, it, 0);
      if (it + 1 < ntile) {  // next scores first: they are computed while the softmax of tile `it` runs
        ok = mbar_wait(&bar_fullk[(it + 1) % kStages], ((it + 1) / kStages) & 1);
        if (!ok) break;
        TC_STAMP(1, it, 1);
        tc_fence_after();
        mma_qk((it + 1) % kStages, (it + 1) & 1);
        TC_STAMP(1, it, 2);
      }
      ok = mbar_wait(&bar_p, it & 1) && mbar_wait(&bar_fullv[it % kStages], (it / kStages) & 1);
      if (!ok) break;
      TC_STAMP(1, it, 3);
      tc_fence_after();
      mma_pv(it % kStages, it == 0);
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
      uint32_t sr[64];
      float mx = -INFINITY;
      TC_STAMP(0, it, 0);
      if (warp_live) {
        if (ok) ok = mbar_wait(&bar_s[buf], (it >> 1) & 1);
        TC_STAMP(0, it, 1);
        if (ok) {
          tc_fence_after();
          tmem_ld32(tmem_s + buf * kBN + lane_sel + half * 64, sr);
          tmem_ld32(tmem_s + buf * kBN + lane_sel + half * 64 + 32, sr + 32);
          tmem_wait_ld();
          TC_STAMP(0, it, 2);
          const int cbase = pos0 + half * 64;
          if (cbase + 64 > L) {  // this thread's 64 columns reach past the prefix: ancestor mask
#pragma unroll
            for (int c = 0; c < 64; ++c) {
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
          for (int c = 0; c < 64; c += 4) {
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
      // P (and O) were last touched by the P V product of tile it-1
      if (warp_live && ok && it >= 1) ok = mbar_wait(&bar_freev[(it - 1) % kStages], ((it - 1) / kStages) & 1);
      TC_STAMP(0, it, 5);
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
        TC_STAMP(0, it, 6);
        // P = 2^((s - m) * scale) as bf16 into the swizzled A-operand buffer; row sum in fp32
        const bool live = m_used > -INFINITY;
        const float neg_ms = live ? -m_used * sc : 0.f;
        float l0 = 0.f, l1 = 0.f;
        unsigned char* prow = smem + kSmemP + half * kRegion;
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8) {
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
          *reinterpret_cast<uint4*>(prow + swz(r, c8)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
        l_run += l0 + l1;
      }
      // V rows past the end of the sequence may hold anything (0 * NaN would poison O): zero them
      if (ok && total - pos0 < kBN) {
        ok = mbar_wait(&bar_fullv[stage], (it / kStages) & 1);  // the tile has landed
        if (ok) {
          const int valid = total - pos0;
          unsigned char* vbase = smem + kSmemV + stage * kTile;
          for (int i = tid; i < (kBN - valid) * 16; i += kSoftmaxThreads) {
            const int rr = valid + (i >> 4), reg = (i >> 3) & 1, c = i & 7;
            *reinterpret_cast<uint4*>(vbase + reg * kRegion + rr * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      }
      TC_STAMP(0, it, 7);
      fence_proxy_async();
      tc_fence_before();
      mbar_arrive(&bar_p);
      TC_STAMP(0, it, 9);
    }
    // epilogue: wait for the last P V; O goes through shared memory (the K/V rings are idle now) so
    // that every global store of a row is one contiguous 512-byte (fp32) or 256-byte (bf16) piece
    TC_MARK(4);
    if (ok) ok = mbar_wait(&bar_freev[(ntile - 1) % kStages], ((ntile - 1) / kStages) & 1);
    TC_MARK(5);
    constexpr int kStageStride = kHD + 4;  // floats per staged row: 16-byte stores stay conflict-free
    float* stage_o = reinterpret_cast<float*>(smem + kSmemK);
    xch[0][half * kBM + r] = l_run;
    if (half == 0) xch[1][r] = m_used * sc * 0.69314718055994531f;  // natural-log units
    if (ok && warp_live) {
      tc_fence_after();
      uint32_t orr[64];
      tmem_ld32(tmem_o + lane_sel + half * 64, orr);
      tmem_ld32(tmem_o + lane_sel + half * 64 + 32, orr + 32);
      tmem_wait_ld();
      float* so = stage_o + r * kStageStride + half * 64;
#pragma unroll
      for (int c4 = 0; c4 < 16; ++c4)
        *reinterpret_cast<float4*>(so + c4 * 4) =
            make_float4(__uint_as_float(orr[c4 * 4]), __uint_as_float(orr[c4 * 4 + 1]), __uint_as_float(orr[c4 * 4 + 2]),
                        __uint_as_float(orr[c4 * 4 + 3]));
    }
    softmax_bar();
    const int rows_here = rows_total - row0 < kBM ? rows_total - row0 : kBM;
    const int wv = warp;  // 0..7: rows wv, wv+8, ... ; lane: columns 4*lane .. 4*lane+3
    if (ok) {
      for (int rr = wv; rr < rows_here; rr += 8) {
        const int grow = row0 + rr, tt = grow / G, hh = kvh * G + grow % G;
        const float4 o4 = *reinterpret_cast<const float4*>(stage_o + rr * kStageStride + lane * 4);
        const float l_tot = xch[0][rr] + xch[0][kBM + rr];
        if (nsplit == 1) {
          const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
          const __nv_bfloat162 a = __floats2bfloat162_rn(o4.x * inv, o4.y * inv), c2 = __floats2bfloat162_rn(o4.z * inv, o4.w * inv);
          uint2 pk;
          pk.x = *reinterpret_cast<const uint32_t*>(&a);
          pk.y = *reinterpret_cast<const uint32_t*>(&c2);
          *reinterpret_cast<uint2*>(p.out + (((size_t)b * p.Ncap + tt) * p.Hq + hh) * kHD + lane * 4) = pk;
        } else {
          const size_t pr = (((size_t)b * p.Hq + hh) * p.Ncap + tt) * p.nsplit_max + split;
          __stcg(reinterpret_cast<float4*>(p.part_o + pr * kHD + lane * 4), o4);
          if (lane == 0) {
            __stcg(p.part_ml + pr * 2, xch[1][rr]);
            __stcg(p.part_ml + pr * 2 + 1, l_tot);
          }
        }
      }
    }
    if (nsplit > 1) {
      // the last split of this row block to finish merges the partials (ticket; nothing spins)
      __threadfence();
      softmax_bar();
      if (tid == 0) {
        int32_t* cnt = p.ticket + ((size_t)b * p.Hkv + kvh) * p.nrb + rb;
        const int t = atomicAdd(cnt, 1);
        last_s = (t == nsplit - 1);
        if (t == nsplit - 1) *cnt = 0;
        __threadfence();
      }
      softmax_bar();
      if (last_s) TC_CTA_LOG(3, gtimer());
      if (last_s) {
        // every lane keeps up to 16 loads in flight (two rows x up to kMaxSplit splits): the merge is
        // bound by L2 latency, not by bytes
        for (int rr = wv; rr < rows_here; rr += 16) {
          float4 acc[2];
          float inv[2];
          size_t orow[2];
          float4 v[2][kMaxSplit];
          float wgt[2];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int r2 = rr + 8 * u;
            const bool on = r2 < rows_here;
            const int grow = row0 + (on ? r2 : rr), tt = grow / G, hh = kvh * G + grow % G;
            const size_t pr = (((size_t)b * p.Hq + hh) * p.Ncap + tt) * p.nsplit_max;
            orow[u] = (((size_t)b * p.Ncap + tt) * p.Hq + hh) * kHD;
            float ms = -INFINITY, ls = 0.f;  // lane s holds split s's (max, sum)
            if (lane < nsplit) {
              ms = __ldcg(p.part_ml + (pr + lane) * 2);
              ls = __ldcg(p.part_ml + (pr + lane) * 2 + 1);
            }
#pragma unroll
            for (int s2 = 0; s2 < kMaxSplit; ++s2)
              v[u][s2] = s2 < nsplit ? __ldcg(reinterpret_cast<const float4*>(p.part_o + (pr + s2) * kHD + lane * 4))
                                     : make_float4(0.f, 0.f, 0.f, 0.f);
            float M = ms;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
            wgt[u] = ms > -INFINITY ? expf(ms - M) : 0.f;
            float lsum = ls * wgt[u];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
            inv[u] = lsum > 0.f ? 1.f / lsum : 0.f;
          }
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int s2 = 0; s2 < kMaxSplit; ++s2) {
              const float w = __shfl_sync(0xffffffffu, wgt[u], s2);
              acc[u].x += v[u][s2].x * w;
              acc[u].y += v[u][s2].y * w;
              acc[u].z += v[u][s2].z * w;
              acc[u].w += v[u][s2].w * w;
            }
            if (rr + 8 * u < rows_here) {
              const __nv_bfloat162 a = __floats2bfloat162_rn(acc[u].x * inv[u], acc[u].y * inv[u]),
                                   c2 = __floats2bfloat162_rn(acc[u].z * inv[u], acc[u].w * inv[u]);
              uint2 pk;
              pk.x = *reinterpret_cast<const uint32_t*>(&a);
              pk.y = *reinterpret_cast<const uint32_t*>(&c2);
              *reinterpret_cast<uint2*>(p.out + orow[u] + lane * 4) = pk;
            }
          }
        }
      }
    }
  }
  TC_MARK(6);
  tc_fence_before();
  __syncthreads();
  TC_MARK(7);
  TC_CTA_LOG(1, gtimer());
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols));
  }
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
  // no tree of this context has more than total_token nodes: row blocks past that are never launched
  const int Nmax = c->cfg.total_token < Ncap ? c->cfg.total_token : Ncap;
  const int nrb = (Nmax * G + kBM - 1) / kBM;
  const int max_pos = page_size == 0 ? seq_capacity : seq_capacity * page_size;
  const int max_tiles = (max_pos + kBN - 1) / kBN;
  // upper bound of the KV splits; the kernel picks the actual number from the device-side sizes
  int nsplit_max = (4 * c->num_sms + B * Hkv - 1) / (B * Hkv);
  if (nsplit_max > max_tiles) nsplit_max = max_tiles;
  if (nsplit_max > kMaxSplit) nsplit_max = kMaxSplit;
  if (nsplit_max < 1) nsplit_max = 1;
  TcParams p;
  p.q = (const __nv_bfloat16*)q; p.out = (__nv_bfloat16*)out;
  p.B = B; p.Ncap = Ncap; p.Nmax = Nmax; p.Hq = Hq; p.Hkv = Hkv; p.G = G; p.page_size = page_size;
  p.seq_capacity = seq_capacity; p.num_pages = num_pages; p.words = c->words; p.nsplit_max = nsplit_max;
  p.num_sms = c->num_sms; p.nrb = nrb;
  p.page_table = page_table; p.kv_len = kv_len; p.n_tree = n_tree; p.anc = anc;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.part_o = nullptr; p.part_ml = nullptr; p.ticket = nullptr; p.st = c->state;
  *status = CAST_OK;
  if (nsplit_max > 1) {
    const size_t rows = (size_t)B * Hq * Ncap * nsplit_max;
    const size_t tickets = (size_t)B * Hkv * nrb;
    const size_t need = rows * (kHD + 2) * sizeof(float) + tickets * sizeof(int32_t);
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
    p.ticket = reinterpret_cast<int32_t*>(p.part_ml + rows * 2);
    // tickets start at zero (every merge also leaves its ticket at zero again)
    if (cudaMemsetAsync(p.ticket, 0, tickets * sizeof(int32_t), stream) != cudaSuccess) {
      *status = CAST_ERR_CUDA;
      return true;
    }
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
  *status = launch_status();
  return true;
}

}  // namespace cast
