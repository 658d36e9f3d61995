// Tensor-core path of cast_tree_attention for bf16, head_dim 128 (sm_100a: tcgen05 + TMEM + TMA).
//
// One CTA owns (sequence b, kv-head, block of 128 query rows, KV split). A query row is a
// (tree token, head of the GQA group) pair, so every K/V tile is fetched once for all tree
// tokens and all heads of the group. Tiles are 64 positions; a CTA needs 112 KB of shared memory
// (Q 32 KB, a ring of three K tiles, a ring of two V tiles) and 256 TMEM columns (two score
// buffers of 64, the output accumulator of 128), so two CTAs share an SM: while one waits for a
// tile or runs its prologue/epilogue, the other streams (128 registers per thread for that). Roles:
//   TMA producers: one warp loads the K tiles, another the V tiles (128B-swizzled, two 64-column
//                  halves each) into the two rings; a K stage is released as soon as Q K^T has
//                  consumed it, a V stage after P V. (One warp for both rings stalled the K loads
//                  behind waits for V stages: the paged batch-64 case went from 142 to 114 us with two.)
//   MMA issuer   : (the whole warp runs the issue loop converged; every MMA / commit elects its one thread)
//                  S = Q K^T by tcgen05.mma (M=128 rows, N=64 positions, K=128) into one of two
//                  TMEM buffers; once the softmax warps have written P, O += P V with P taken
//                  from tensor memory (A operand in TMEM) and V as the MN-major B operand: used
//                  exactly as it lies in the cache, no transpose. Q K^T of tile i+1 is issued
//                  before P of tile i is awaited.
//   4 softmax warps: one thread per query row reads its 64 scores with tcgen05.ld, applies the
//                  prefix/ancestor mask (only tiles that reach past the prefix need one) and
//                  writes P = 2^((s - m) * scale) as bf16 over the scores, in tensor memory
//                  (tcgen05.st). Every tile takes one pass: the row's reference m starts at 0 and
//                  moves (by a power of two, O in TMEM rescaled with it) only when a row's P would
//                  leave the range 2^-60 .. 2^60.
// The kernel is launched in thread-block clusters: a cluster covers the row blocks of one
// (sequence, kv-head) and splits each one's KV range over its CTAs, the number of splits per row
// block being decided on the device from the actual tree size (the host only knows the largest
// tree). The splits of a row block are merged through distributed shared memory: every CTA stages
// its partial output in its own shared memory, the cluster meets at a barrier, and each CTA
// combines and writes its share of the rows, reading its peers' partials directly. Nothing goes
// through global memory and nothing spins. All mbarrier waits are bounded: on expiry the CTA
// records CAST_ERR_TIMEOUT, contributes nothing to the merge, and still meets its cluster.
#include <cuda.h>
#include <cuda_fp16.h>
#include <math.h>

#include "cast_internal.h"


namespace cast {

namespace {

constexpr int kBM = 128;          // query rows per CTA (UMMA M)
constexpr int kBN = 64;           // positions per tile
constexpr int kHD = 128;          // head dim
constexpr int kStagesK = 3;       // tiles in the K ring
constexpr int kStagesV = 2;       // tiles in the V ring
constexpr int kSoftmaxThreads = 128;               // one thread per query row
constexpr int kThreadsTC = 256;  // 4 softmax warps, K producer, MMA issuer, V producer, 1 idle: registers are allotted per 4 warps
constexpr int kRegionQ = kBM * 128;                // [128 rows][64] bf16, 128-byte rows: 16 KB
constexpr int kRegionKV = kBN * 128;               // [64 positions][64] bf16: 8 KB
constexpr int kTileKV = 2 * kRegionKV;             // a [64][128] K or V tile: 16 KB
constexpr int kSmemQ = 0;                          // 2 regions (d 0-63, d 64-127)
constexpr int kSmemK = 2 * kRegionQ;                 // kStagesK tiles
constexpr int kSmemV = kSmemK + kStagesK * kTileKV;  // kStagesV tiles
constexpr int kSmemBar = kSmemV + kStagesV * kTileKV;  // mbarriers and two words, 128 bytes
constexpr int kSmemBytes = kSmemBar + 128;           // 112 KB + 128 B: two CTAs per SM
constexpr int kTmemCols = 256;                     // S0: [0,64), S1: [64,128), O: [128,256)
constexpr long long kWaitCycles = 4000000000ll;    // about two seconds
constexpr int kMaxSplit = 8;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  int B, Ncap, Nmax, Hq, Hkv, G, page_size, seq_capacity, num_pages, words;
  int q_tma;  // Q row blocks are fetched by TMA (the group size divides 128)
  const int32_t* worklist;  // one decoded work item per CTA (8 ints each), or null: every CTA decodes for itself
  int early;  // the tree arrays, lengths, page table and prefix rows may be read before the dependency wait
  int cs;   // CTAs per cluster (1..8); 0: no clusters, splits sized on the device and merged through global memory
  int rpc;  // cluster mode: row blocks a cluster covers at most (cs is a multiple of it)
  int nsplit_max, num_sms, nrb;  // global-merge mode
  __half* part_o;    // [B][Hq][Ncap][nsplit_max][D]: partial rows normalised by their own sum, half precision
  float* part_ml;    // [B][Hq][Ncap][nsplit_max][2]
  int32_t* ticket;   // [B][Hkv][nrb]
  const int32_t* page_table;
  const int32_t* kv_len;
  const int32_t* n_tree;
  const int32_t* first_row;  // [B] or null: output rows start at this tree token (the tokens before it are context only)
  const uint32_t* anc;
  float scale_log2;
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
// The MMA and commit wrappers are called by all 32 lanes of the issuing warp, converged, and elect the one
// thread that issues inside: the operands are then warp-uniform values computed in convergent code, which the
// compiler can keep in uniform registers. (Computed inside an `if (lane == 0)` block they took a chain of
// vector-to-uniform moves per instruction: about 100 cycles per MMA, which made the issuing warp the
// bottleneck of the tile loop.)
// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulation.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "elect.sync _|q, 0xffffffff;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]: the A operand (128 rows, one per TMEM lane; 16 bf16 of the K extent
// packed two to a 32-bit column, 8 columns per instruction) comes from tensor memory.
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "elect.sync _|q, 0xffffffff;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile(
      "{\n\t.reg .pred q;\n\t"
      "elect.sync _|q, 0xffffffff;\n\t"
      "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(smem_u32(bar))
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
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// Packed fp32 pairs (one instruction, two lanes of the FMA pipe): the softmax's inner loop is bound by
// instruction issue, and its multiply-add and its running sum pair up naturally.
__device__ __forceinline__ unsigned long long pack_f2(float a, float b) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack_f2(unsigned long long v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma_f2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ unsigned long long add_f2(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Waits for this thread's tensor-memory loads and ties the wait to the registers they fill, so that no use of
// them can be scheduled above it (a load may be issued long before its values are needed).
__device__ __forceinline__ void tmem_wait_ld_regs(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),
                 "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
                 "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}
// One half tile (32 scores of this thread's row, in registers) of the single-pass softmax: P = 2^(s * scale -
// m * scale) as bf16 pairs, the row sum as a packed pair of partial sums. kMasked: `vv` holds the 32 visibility bits.
template <bool kMasked>
__device__ __forceinline__ void softmax_half(const uint32_t (&sr)[32], unsigned long long sc2, unsigned long long neg2,
                                             uint32_t vv, unsigned long long& lacc, uint32_t (&pk)[16]) {
#pragma unroll
  for (int e = 0; e < 16; ++e) {
    const int c = 2 * e;
    float x0, x1;
    unpack_f2(fma_f2(pack_f2(__uint_as_float(sr[c]), __uint_as_float(sr[c + 1])), sc2, neg2), x0, x1);
    float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
    if (kMasked) {
      p0 = ((vv >> c) & 1u) ? p0 : 0.f;
      p1 = ((vv >> (c + 1)) & 1u) ? p1 : 0.f;
    }
    lacc = add_f2(lacc, pack_f2(p0, p1));
    const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
    pk[e] = *reinterpret_cast<const uint32_t*>(&pb);
  }
}

// 32 bits of the visibility vector of one query row, starting at tree index `start` (which may be
// negative: prefix positions, always visible; or past the tree: never visible). aw = the row's
// ancestor mask (bits >= n_tree are zero).
__device__ __forceinline__ uint32_t vis_word(const uint32_t (&aw)[4], int i) {
  return i < 0 ? 0xffffffffu : i == 0 ? aw[0] : i == 1 ? aw[1] : i == 2 ? aw[2] : i == 3 ? aw[3] : 0u;
}
__device__ __forceinline__ uint32_t vis_bits32(const uint32_t (&aw)[4], int start) {
  const int wi = start >> 5, sh = start & 31;  // arithmetic shift: floor division for negative starts
  const uint32_t lo = vis_word(aw, wi), hi = vis_word(aw, wi + 1);
  return sh == 0 ? lo : ((lo >> sh) | (hi << (32 - sh)));
}

// Byte offset of 16-byte chunk `c` (0..7) of row `r` inside a 128B-swizzled [rows][64 bf16] region.
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

__device__ __forceinline__ int clampi(int x, int lo, int hi) { return x < lo ? lo : (x > hi ? hi : x); }

// The grid is one-dimensional and launched in clusters of p.cs CTAs. A cluster takes one
// (sequence, kv-head, group of up to p.rpc row blocks); its CTAs share the group's row blocks and
// split each one's KV range evenly: with nr row blocks actually present (known only on the device,
// from n_tree), every row block gets cs / nr splits. A small tree under a large token budget thus
// turns the CTAs reserved for its absent row blocks into extra KV splits. Clusters are enumerated on
// the device from the actual sizes, sequences with the longest pieces first (the block scheduler
// hands clusters out in index order, so the long pieces start first and the short ones fill the
// gaps), the kv-head running fastest so that the heads of one sequence stream the same pages at the
// same time. Clusters past the count exit at once. Every warp computes the same values (all 32
// lanes must call).
struct WorkItem {
  int b, kvh, rb, split, nsplit, N, L, F;
  bool valid;   // the cluster has work
  bool active;  // this CTA has a row block (an inactive CTA of a valid cluster only keeps the barriers in step)
};

__device__ __forceinline__ WorkItem decode_work(const TcParams& p, int cid, int crank) {
  constexpr int KB = CAST_MAX_BATCH / 32;
  const int lane = threadIdx.x & 31;
  const int max_pos = p.page_size == 0 ? p.seq_capacity : p.seq_capacity * p.page_size;
  int Nv[KB], Lv[KB], Fv[KB], tl[KB], nr[KB], cnt[KB], off[KB];
#pragma unroll
  for (int k = 0; k < KB; ++k) {  // all loads first: one memory round trip
    const int bb = k * 32 + lane;
    Nv[k] = bb < p.B ? p.n_tree[bb] : 0;
    Lv[k] = bb < p.B ? p.kv_len[bb] : 0;
    Fv[k] = (p.first_row != nullptr && bb < p.B) ? p.first_row[bb] : 0;
  }
#pragma unroll
  for (int k = 0; k < KB; ++k) {
    Nv[k] = clampi(Nv[k], 0, p.Nmax);
    Fv[k] = clampi(Fv[k], 0, Nv[k]);
    Lv[k] = Lv[k] < 0 ? 0 : Lv[k];
    int total = Lv[k] + Nv[k];
    total = total > max_pos ? max_pos : total;
    nr[k] = ((Nv[k] - Fv[k]) * p.G + kBM - 1) / kBM;
    tl[k] = nr[k] > 0 ? (total + kBN - 1) / kBN : 0;
    cnt[k] = p.Hkv * ((nr[k] + p.rpc - 1) / p.rpc);
    off[k] = 0;
  }
  if (p.B > 1) {
#pragma unroll 8
    for (int j = 0; j < p.B; ++j) {  // sequence j precedes sequence b when it is longer, ties by index
      const int src = j & 31;
      int pj, cj;
      if (j < 32) {
        pj = __shfl_sync(0xffffffffu, tl[0], src);
        cj = __shfl_sync(0xffffffffu, cnt[0], src);
      } else {
        pj = __shfl_sync(0xffffffffu, tl[KB - 1], src);
        cj = __shfl_sync(0xffffffffu, cnt[KB - 1], src);
      }
#pragma unroll
      for (int k = 0; k < KB; ++k) {
        const int bm = k * 32 + lane;
        if (pj > tl[k] || (pj == tl[k] && j < bm)) off[k] += cj;
      }
    }
  }
  WorkItem w;
  w.valid = w.active = false;
  w.b = w.kvh = w.rb = w.split = w.N = w.L = w.F = 0;
  w.nsplit = 1;
#pragma unroll
  for (int k = 0; k < KB; ++k) {
    const unsigned hit = __ballot_sync(0xffffffffu, cid >= off[k] && cid < off[k] + cnt[k]);
    if (hit != 0u && !w.valid) {
      const int bl = __ffs(hit) - 1;
      const int local = cid - __shfl_sync(0xffffffffu, off[k], bl);
      const int nrb = __shfl_sync(0xffffffffu, nr[k], bl);
      w.N = __shfl_sync(0xffffffffu, Nv[k], bl);
      w.F = __shfl_sync(0xffffffffu, Fv[k], bl);
      w.L = __shfl_sync(0xffffffffu, Lv[k], bl);
      w.b = k * 32 + bl;
      w.kvh = local % p.Hkv;
      const int grp = local / p.Hkv;
      int nr_in = nrb - grp * p.rpc;
      nr_in = nr_in > p.rpc ? p.rpc : nr_in;  // >= 1 for an enumerated group
      w.nsplit = p.cs / nr_in;
      const int rbl = crank / w.nsplit;
      w.split = crank % w.nsplit;
      w.rb = grp * p.rpc + rbl;
      w.active = rbl < nr_in;
      w.valid = true;
    }
  }
  return w;
}

// ---- cluster primitives
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
  return v;
}

constexpr int kStageStride = kHD + 4;   // floats per staged output row: 16-byte accesses stay conflict-free
constexpr int kStageStrideH = kHD + 8;  // halves per staged row of a cluster-merged partial (272 bytes)
__device__ __forceinline__ uint2 ld_cluster_u2(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared::cluster.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}

// Merge of the splits of a row block through distributed shared memory. Every CTA of the split
// group has staged its partial output rows, normalised by their own sum and rounded to half precision
// (the merge moves half the bytes that way; the rounding, 2^-11 relative, is a quarter of the bf16
// output's), and (max, sum) per row in its own shared memory. This CTA owns the rows rr with
// rr % nsplit == split and reads them from all peers: split s weighs sum_s * e^(max_s - max).
// Warp w takes owned rows w, w+8, ...; a lane owns 4 output columns; ROWS x SPL loads in flight.
template <int ROWS, int SPL>
__device__ __forceinline__ void merge_rows(const TcParams& p, uint32_t stage_o_s, uint32_t stage_ml_s, int rank0,
                                           int b, int kvh, int row0, int rows_here, int nsplit, int split) {
  const int lane = threadIdx.x & 31, wv = threadIdx.x >> 5, G = p.G;
  const int owned = rows_here > split ? (rows_here - split + nsplit - 1) / nsplit : 0;
  for (int i0 = wv; i0 < owned; i0 += 8 * ROWS) {
    uint2 v[ROWS][SPL];
    float wgt[ROWS], inv[ROWS];
    size_t orow[ROWS];
#pragma unroll
    for (int u = 0; u < ROWS; ++u) {
      const int i2 = i0 + 8 * u;
      const int rr = split + nsplit * (i2 < owned ? i2 : i0);
      const int grow = row0 + rr, tt = grow / G, hh = kvh * G + grow % G;
      orow[u] = (((size_t)b * p.Ncap + tt) * p.Hq + hh) * kHD;
      float ms = -INFINITY, ls = 0.f;  // lane s holds split s's (max, sum)
      if (lane < nsplit) {
        const float2 ml = ld_cluster_f2(map_to_rank(stage_ml_s + (uint32_t)rr * 8u, (uint32_t)(rank0 + lane)));
        ms = ml.x;
        ls = ml.y;
      }
#pragma unroll
      for (int s2 = 0; s2 < SPL; ++s2)
        v[u][s2] = s2 < nsplit ? ld_cluster_u2(map_to_rank(stage_o_s + (uint32_t)(rr * kStageStrideH + lane * 4) * 2u,
                                                           (uint32_t)(rank0 + s2)))
                               : make_uint2(0u, 0u);
      float M = ms;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
      wgt[u] = ms > -INFINITY ? ls * expf(ms - M) : 0.f;
      float lsum = wgt[u];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
      inv[u] = lsum > 0.f ? 1.f / lsum : 0.f;
    }
#pragma unroll
    for (int u = 0; u < ROWS; ++u) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int s2 = 0; s2 < SPL; ++s2) {
        const float w = __shfl_sync(0xffffffffu, wgt[u], s2);
        if (w > 0.f) {  // a split without visible positions staged nothing: its buffer may hold anything
          const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&v[u][s2].x));
          const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&v[u][s2].y));
          acc.x += lo.x * w;
          acc.y += lo.y * w;
          acc.z += hi.x * w;
          acc.w += hi.y * w;
        }
      }
      if (i0 + 8 * u < owned) {
        const __nv_bfloat162 a = __floats2bfloat162_rn(acc.x * inv[u], acc.y * inv[u]),
                             c2 = __floats2bfloat162_rn(acc.z * inv[u], acc.w * inv[u]);
        uint2 pk;
        pk.x = *reinterpret_cast<const uint32_t*>(&a);
        pk.y = *reinterpret_cast<const uint32_t*>(&c2);
        *reinterpret_cast<uint2*>(p.out + orow[u] + lane * 4) = pk;
      }
    }
  }
}

// ---- global-merge mode -------------------------------------------------------------------------
// For launches with long CTAs or many ragged sequences, where an even load matters more than the
// cost of the merge: no clusters; CTA i takes work item i. Sequence b has Hkv * row_blocks(b) *
// splits(b) items, splits(b) = ceil(tiles(b) / chunk), chunk (>= 4 tiles) being the smallest piece
// size for which all items fit into the launched waves of 2 * num_sms CTAs; when the unsplit work
// already fills a wave, nothing is split. The pieces are of about equal size whatever the mix of
// lengths. Partials go to a workspace; the last CTA of a row block to finish (an atomic ticket,
// nothing spins) merges them.
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ WorkItem decode_work_chunked(const TcParams& p, int idx, int grid) {
  constexpr int KB = CAST_MAX_BATCH / 32;
  const int lane = threadIdx.x & 31;
  const int max_pos = p.page_size == 0 ? p.seq_capacity : p.seq_capacity * p.page_size;
  int Nv[KB], Lv[KB], Fv[KB], tl[KB], nr[KB];
#pragma unroll
  for (int k = 0; k < KB; ++k) {  // all loads first: one memory round trip
    const int bb = k * 32 + lane;
    Nv[k] = bb < p.B ? p.n_tree[bb] : 0;
    Lv[k] = bb < p.B ? p.kv_len[bb] : 0;
    Fv[k] = (p.first_row != nullptr && bb < p.B) ? p.first_row[bb] : 0;
  }
  int base = 0, T = 0, tmax = 0;
#pragma unroll
  for (int k = 0; k < KB; ++k) {
    Nv[k] = clampi(Nv[k], 0, p.Nmax);
    Fv[k] = clampi(Fv[k], 0, Nv[k]);
    Lv[k] = Lv[k] < 0 ? 0 : Lv[k];
    int total = Lv[k] + Nv[k];
    total = total > max_pos ? max_pos : total;
    nr[k] = ((Nv[k] - Fv[k]) * p.G + kBM - 1) / kBM;
    tl[k] = nr[k] > 0 ? (total + kBN - 1) / kBN : 0;
    base += p.Hkv * nr[k];
    T += p.Hkv * nr[k] * tl[k];
    tmax = tl[k] > tmax ? tl[k] : tmax;
  }
  base = warp_sum(base);
  T = warp_sum(T);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tmax = max(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
  const int slots = 2 * p.num_sms;
  int W = (base + slots - 1) / slots;
  W = W < 1 ? 1 : W;
  int cap = W * slots;
  cap = cap > grid ? grid : cap;
  // smallest chunk (>= 4 tiles) whose item count fits: the count falls as the chunk grows, and a chunk
  // of tmax tiles (no splits at all) always fits
  auto items_at = [&](int chunk) {
    int items = 0;
#pragma unroll
    for (int k = 0; k < KB; ++k) {
      int n = (tl[k] + chunk - 1) / chunk;
      n = n > p.nsplit_max ? p.nsplit_max : n;
      items += p.Hkv * nr[k] * n;
    }
    return warp_sum(items);
  };
  int lo = (T + cap - 1) / cap, hi = tmax < 4 ? 4 : tmax;
  lo = lo < 4 ? 4 : lo;
  lo = lo > hi ? hi : lo;
  if (base >= slots) lo = hi;  // the unsplit work fills a wave already: no splits
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (items_at(mid) <= cap) hi = mid; else lo = mid + 1;
  }
  const int chunk = lo;
  int ns[KB], cnt[KB], off[KB];
#pragma unroll
  for (int k = 0; k < KB; ++k) {
    int n = (tl[k] + chunk - 1) / chunk;
    n = n > p.nsplit_max ? p.nsplit_max : n;
    ns[k] = n < 1 ? 1 : n;
    cnt[k] = p.Hkv * nr[k] * ns[k];
    off[k] = 0;
  }
  // items are numbered longest piece first (the block scheduler hands CTAs out in index order, so
  // the long pieces start first and the short ones fill the gaps): sequence j precedes sequence b
  // when its pieces are longer, ties by index
  int key[KB];
#pragma unroll
  for (int k = 0; k < KB; ++k) key[k] = tl[k] * 16 / ns[k];
  if (p.B > 1) {
#pragma unroll 8
    for (int j = 0; j < p.B; ++j) {
      const int src = j & 31;
      int pj, cj;
      if (j < 32) {
        pj = __shfl_sync(0xffffffffu, key[0], src);
        cj = __shfl_sync(0xffffffffu, cnt[0], src);
      } else {
        pj = __shfl_sync(0xffffffffu, key[KB - 1], src);
        cj = __shfl_sync(0xffffffffu, cnt[KB - 1], src);
      }
#pragma unroll
      for (int k = 0; k < KB; ++k) {
        const int bm = k * 32 + lane;
        if (pj > key[k] || (pj == key[k] && j < bm)) off[k] += cj;
      }
    }
  }
  WorkItem w;
  w.valid = w.active = false;
  w.b = w.kvh = w.rb = w.split = w.N = w.L = w.F = 0;
  w.nsplit = 1;
#pragma unroll
  for (int k = 0; k < KB; ++k) {
    const unsigned hit = __ballot_sync(0xffffffffu, idx >= off[k] && idx < off[k] + cnt[k]);
    if (hit != 0u && !w.valid) {
      const int bl = __ffs(hit) - 1;
      const int local = idx - __shfl_sync(0xffffffffu, off[k], bl);
      w.nsplit = __shfl_sync(0xffffffffu, ns[k], bl);
      w.N = __shfl_sync(0xffffffffu, Nv[k], bl);
      w.F = __shfl_sync(0xffffffffu, Fv[k], bl);
      w.L = __shfl_sync(0xffffffffu, Lv[k], bl);
      w.b = k * 32 + bl;
      w.kvh = local % p.Hkv;
      const int rest = local / p.Hkv;
      w.split = rest % w.nsplit;
      w.rb = rest / w.nsplit;
      w.valid = w.active = true;
    }
  }
  return w;
}

// Merge of the split partials of a row block, run by all 8 warps of the last CTA to finish it.
// Warp w takes rows w, w+8, ...; a lane owns 4 output columns. ROWS rows x SPL splits = 16 loads are
// in flight per lane: the merge is bound by L2 latency, not by bytes.
template <int ROWS, int SPL>
__device__ __forceinline__ void merge_rows_global(const TcParams& p, int b, int kvh, int row0, int rows_here, int nsplit) {
  const int lane = threadIdx.x & 31, wv = threadIdx.x >> 5, G = p.G;
  for (int rr = wv; rr < rows_here; rr += 8 * ROWS) {
    uint2 v[ROWS][SPL];
    float wgt[ROWS], inv[ROWS], msv[ROWS], lsv[ROWS];
    size_t orow[ROWS];
    // every load of every row first, then the reductions (a reduction waits for its row's loads; with the next
    // row's loads issued behind it the rows cost one round trip to L2 each, 6-7 us for eight)
#pragma unroll
    for (int u = 0; u < ROWS; ++u) {
      const int r2 = rr + 8 * u;
      const int grow = row0 + (r2 < rows_here ? r2 : rr), tt = grow / G, hh = kvh * G + grow % G;
      const size_t pr = (((size_t)b * p.Hq + hh) * p.Ncap + tt) * p.nsplit_max;
      orow[u] = (((size_t)b * p.Ncap + tt) * p.Hq + hh) * kHD;
      msv[u] = -INFINITY;  // lane s holds split s's (max, sum)
      lsv[u] = 0.f;
      if (lane < nsplit) {
        const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + (pr + lane) * 2));
        msv[u] = ml.x;
        lsv[u] = ml.y;
      }
#pragma unroll
      for (int s2 = 0; s2 < SPL; ++s2)
        v[u][s2] = s2 < nsplit ? __ldcg(reinterpret_cast<const uint2*>(p.part_o + (pr + s2) * kHD + lane * 4))
                               : make_uint2(0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < ROWS; ++u) {
      const float ms = msv[u], ls = lsv[u];
      float M = ms;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
      wgt[u] = ms > -INFINITY ? ls * expf(ms - M) : 0.f;  // split s weighs sum_s * e^(max_s - max)
      float lsum = wgt[u];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
      inv[u] = lsum > 0.f ? 1.f / lsum : 0.f;
    }
#pragma unroll
    for (int u = 0; u < ROWS; ++u) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int s2 = 0; s2 < SPL; ++s2) {
        const float w = __shfl_sync(0xffffffffu, wgt[u], s2);
        if (w > 0.f) {  // a split without visible positions wrote zeros at best
          const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&v[u][s2].x));
          const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&v[u][s2].y));
          acc.x += lo.x * w;
          acc.y += lo.y * w;
          acc.z += hi.x * w;
          acc.w += hi.y * w;
        }
      }
      if (rr + 8 * u < rows_here) {
        const __nv_bfloat162 a = __floats2bfloat162_rn(acc.x * inv[u], acc.y * inv[u]),
                             c2 = __floats2bfloat162_rn(acc.z * inv[u], acc.w * inv[u]);
        uint2 pk;
        pk.x = *reinterpret_cast<const uint32_t*>(&a);
        pk.y = *reinterpret_cast<const uint32_t*>(&c2);
        *reinterpret_cast<uint2*>(p.out + orow[u] + lane * 4) = pk;
      }
    }
  }
}

// One work item as eight ints: {b | kvh << 8 | rb << 16 | valid << 24 | active << 25, split | nsplit << 16, N, L, F, 0, 0, 0}
__device__ __forceinline__ void store_item(int32_t* dst, const WorkItem& w) {
  dst[0] = w.b | (w.kvh << 8) | (w.rb << 16) | ((w.valid ? 1 : 0) << 24) | ((w.active ? 1 : 0) << 25);
  dst[1] = w.split | (w.nsplit << 16);
  dst[2] = w.N;
  dst[3] = w.L;
  dst[4] = w.F;
}
__device__ __forceinline__ WorkItem load_item(const int32_t* src) {
  const int4 a = *reinterpret_cast<const int4*>(src);
  const int f = src[4];
  WorkItem w;
  w.b = a.x & 0xff; w.kvh = (a.x >> 8) & 0xff; w.rb = (a.x >> 16) & 0xff;
  w.valid = ((a.x >> 24) & 1) != 0; w.active = ((a.x >> 25) & 1) != 0;
  w.split = a.y & 0xffff; w.nsplit = a.y >> 16;
  w.N = a.z; w.L = a.w; w.F = f;
  return w;
}
// The work decode of every CTA of a launch, done once: warp i decodes what CTA i would decode for itself.
__global__ void __launch_bounds__(256) attn_worklist_kernel(const TcParams p, int grid, int32_t* list) {
  const int idx = (int)blockIdx.x * 8 + (int)(threadIdx.x >> 5);
  if (idx >= grid) return;
  const WorkItem w = p.cs == 0 ? decode_work_chunked(p, idx, grid) : decode_work(p, idx / p.cs, idx % p.cs);
  if ((threadIdx.x & 31) == 0) store_item(list + (size_t)idx * 8, w);
}

__global__ void __launch_bounds__(kThreadsTC, 2)
tree_attn_tc_kernel(const TcParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                    const __grid_constant__ CUtensorMap map_q) {
  extern __shared__ __align__(1024) unsigned char smem[];  // no static shared memory: the base is 1 KB aligned

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cs = p.cs;
  const int crank = cs > 1 ? (int)cluster_ctarank() : 0;
  if (warp == 4 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_q)) : "memory");
  }
  // Programmatic dependent launch: this grid may become resident while the previous kernel of the
  // stream drains; nothing written by earlier kernels is read before this point. (No-ops for a plain launch.)
  // In the default mode nothing is read before the wait. In "early" mode (a promise of the caller, see
  // cast_set_attention_early_reads) only Q and the cache rows of the tree tokens can come from the previous
  // kernel: the work decode, the ancestor masks, the page ids and the K/V tiles that lie wholly inside the
  // prefix are fetched while that kernel still runs, and every warp waits just before the first thing it does
  // that depends on it (the Q load, a tile that reaches the tree rows, the output rows). The dependents are
  // released only after this CTA's own wait, so "everything before my predecessor is complete" keeps holding
  // down the chain.
  const bool early = p.early != 0;
  if (!early) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  const WorkItem wk = p.worklist != nullptr ? load_item(p.worklist + (size_t)blockIdx.x * 8)
                      : cs == 0            ? decode_work_chunked(p, (int)blockIdx.x, (int)gridDim.x)
                                           : decode_work(p, (int)blockIdx.x / cs, crank);
  if (blockIdx.x < p.B && tid == 0 && p.n_tree[blockIdx.x] > p.Nmax) report(p.st, CAST_ERR_BAD_TREE, blockIdx.x);
  if (!wk.valid) return;  // the whole cluster leaves (a CTA that exits counts as having released its dependents)
  const int b = wk.b, kvh = wk.kvh, rb = wk.rb, split = wk.split, N = wk.N, L = wk.L;
  const int nsplit = wk.nsplit;
  const int G = p.G, F = wk.F, rows_total = (N - F) * G, row0 = rb * kBM;
  const int grow0 = F * G + row0;  // the row block's first row counted from tree token 0
  const int max_pos = p.page_size == 0 ? p.seq_capacity : p.seq_capacity * p.page_size;
  int total = L + N;
  if (total > max_pos) {
    if (tid == 0) report(p.st, CAST_ERR_BAD_PAGE, b);
    total = max_pos;
  }
  const int ntiles = (total + kBN - 1) / kBN;  // >= 1 because N >= 1 here
  float* stage_o = reinterpret_cast<float*>(smem + kSmemK);   // [128][kStageStride] floats < K ring + V ring + P
  float* stage_ml = reinterpret_cast<float*>(smem + kSmemQ);  // [128][2]
  const bool aligned = (smem_u32(smem) & 1023u) == 0u;  // the swizzled operand regions need a 1 KB aligned base
  if (!wk.active || !aligned) {
    // no row block for this CTA (or an unusable shared-memory base): it contributes nothing, but the
    // other CTAs of the cluster still meet it at both cluster barriers
    if (!aligned && tid == 0) report(p.st, CAST_ERR_CUDA, 1024);
    if (tid < kBM) {
      stage_ml[tid * 2] = -INFINITY;
      stage_ml[tid * 2 + 1] = 0.f;
    }
    if (cs > 1) {
      cluster_sync_all();
      cluster_sync_all();
    }
    return;
  }
  const int t0 = (int)((long long)split * ntiles / nsplit), t1 = (int)((long long)(split + 1) * ntiles / nsplit);
  const int ntile = t1 - t0;
  const int r = tid & (kBM - 1);  // softmax role: the query row of this thread
  const int row = row0 + r;
  const bool row_ok = warp < 4 && row < rows_total;
  const int t_tok = row_ok ? F + row / G : 0, h_q = kvh * G + (row_ok ? row % G : 0);

  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kSmemBar);
  static_assert(kStagesK <= 3 && kStagesV <= 2, "barrier slots");
  uint64_t* bar_fullk = bars;          // [kStagesK]
  uint64_t* bar_fullv = bars + 3;      // [kStagesV]
  uint64_t* bar_freek = bars + 5;      // [kStagesK]
  uint64_t* bar_freev = bars + 8;      // [kStagesV]
  uint64_t* bar_s = bars + 10;         // [2]
  uint64_t* bar_p = bars + 12;         // [2]: tile it uses bar_p[it & 1], phase it >> 1
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(bars + 14);
  int* last_s = reinterpret_cast<int*>(bars + 14) + 1;
  uint64_t* bar_q = bars + 15;         // the Q row block has landed (TMA)

  // ---- producer helper (warp 4; all 32 lanes call it): which = 0: K tile j, which = 1: V tile j
  // Paged caches: a producer warp reads the page table 32 entries at a time (one coalesced load, lane l keeps
  // entry win0 + l) and hands the ids of a tile's pages out by shuffle: one round trip to memory per 32 / (pages
  // per tile) tiles instead of one per tile, which the tile's copies had to wait for.
  int pg_win0 = -0x40000000, pg_id = 0;
  auto issue_tile = [&](int j, int which) -> bool {
    const int stages = which ? kStagesV : kStagesK, stage = j % stages;
    unsigned char* dst = smem + (which ? kSmemV : kSmemK) + stage * kTileKV;
    uint64_t* full = which ? &bar_fullv[stage] : &bar_fullk[stage];
    const CUtensorMap* map = which ? &map_v : &map_k;
    const int pos0 = (t0 + j) * kBN;
    const int ps = p.page_size;
    int npages = 0, page = 0;
    if (ps != 0) {
      const int ppt = kBN / ps, e0 = pos0 / ps;  // the tile's first page-table entry
      npages = (total - pos0 + ps - 1) / ps;
      npages = npages > ppt ? ppt : npages;
      if (e0 < pg_win0 || e0 + ppt > pg_win0 + 32) {  // (warp-uniform)
        pg_win0 = e0;
        pg_id = e0 + lane < p.seq_capacity ? p.page_table[(size_t)b * p.seq_capacity + e0 + lane] : 0;
      }
      const int pg = __shfl_sync(0xffffffffu, pg_id, e0 - pg_win0 + (lane >> 1));
      if (lane < npages * 2) {
        page = pg;
        if (page < 0 || page >= p.num_pages) {
          report(p.st, CAST_ERR_BAD_PAGE, b);
          page = 0;
        }
      }
    }
    if (j >= stages && !mbar_wait(which ? &bar_freev[stage] : &bar_freek[stage], ((j / stages) - 1) & 1)) return false;
    if (ps == 0) {
      if (lane == 0) mbar_expect_tx(full, kTileKV);
      __syncwarp();
      if (lane < 2) tma_load_3d(map, dst + lane * kRegionKV, full, lane * 64, kvh, b * p.seq_capacity + pos0);
    } else {  // at most 8 pages per tile (page size >= 8): one (page, column half) per lane
      if (lane == 0) mbar_expect_tx(full, (uint32_t)npages * ps * 128 * 2);
      __syncwarp();
      if (lane < npages * 2) {
        const int slot = lane >> 1, hsel = lane & 1;
        tma_load_4d(map, dst + hsel * kRegionKV + slot * ps * 128, full, hsel * 64, kvh, 0, page);
      }
    }
    __syncwarp();
    return true;
  };
  // a producer warp fills its ring tile by tile (K: warp 4, V: warp 6); after an expired wait it reports,
  // then waits (bounded) for its copies in flight, which must land before the CTA's shared memory is released
  auto produce = [&](int which, int first, bool waited) {
    const int stages = which ? kStagesV : kStagesK;
    int armed = first;
    bool ok = true;
    for (int j = first; j < ntile && ok; ++j) {
      if (!waited && (t0 + j + 1) * kBN > L) {  // the first tile that reaches the tree tokens' rows
        asm volatile("griddepcontrol.wait;" ::: "memory");
        waited = true;
      }
      ok = issue_tile(j, which);
      if (ok) armed = j + 1;
    }
    if (!waited) asm volatile("griddepcontrol.wait;" ::: "memory");  // (this warp writes output rows in the merge)
    if (!ok) {
      if (lane == 0) report(p.st, CAST_ERR_TIMEOUT, b);
      for (int j = (armed > stages ? armed - stages : 0); j < armed; ++j) {
        const long long tw = clock64();
        while (!mbar_test(which ? &bar_fullv[j % stages] : &bar_fullk[j % stages], (j / stages) & 1) &&
               clock64() - tw < kWaitCycles) {}
      }
    }
  };
  int k_issued = 0;  // K tiles issued before the CTA barrier (they need no stage wait)

  uint32_t aw[4] = {0u, 0u, 0u, 0u};  // softmax role: ancestor mask of this thread's row
  if (warp == 4) {
    if (lane == 0) {
      for (int s = 0; s < kStagesK; ++s) {
        mbar_init(&bar_fullk[s], 1);
        mbar_init(&bar_freek[s], 1);
      }
      for (int s = 0; s < kStagesV; ++s) {
        mbar_init(&bar_fullv[s], 1);
        mbar_init(&bar_freev[s], 1);
      }
      mbar_init(&bar_s[0], 1);
      mbar_init(&bar_s[1], 1);
      mbar_init(&bar_p[0], kSoftmaxThreads);
      mbar_init(&bar_p[1], kSoftmaxThreads);
      mbar_init(bar_q, 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_proxy_async();
    }
    __syncwarp();
    __threadfence_block();
    asm volatile("bar.arrive 2, %0;" ::"n"(kThreadsTC) : "memory");
    // The Q row block: rows are (tree token, head of the group) pairs, so a block is 128 / G consecutive
    // tokens x the group's G heads x 128 dims: one 3-D box per 64-dim half, 128-byte swizzled like K. (Rows
    // past the tree hold whatever the caller's buffer holds: their P is masked to exact zeros.)
    if (early) {  // prefix tiles first, then the wait, then Q (the previous kernel may have written it)
      for (; k_issued < kStagesK && k_issued < ntile && (t0 + k_issued + 1) * kBN <= L; ++k_issued) issue_tile(k_issued, 0);
      asm volatile("griddepcontrol.wait;" ::: "memory");
      asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    if (p.q_tma && ntile > 0) {  // (a split without tiles stages its empty partial in this region right away)
      if (lane == 0) mbar_expect_tx(bar_q, 2 * kRegionQ);
      __syncwarp();
      if (lane < 2)
        tma_load_3d(&map_q, smem + kSmemQ + lane * kRegionQ, bar_q, lane * 64, kvh * G, b * p.Ncap + F + row0 / G);
    }
    // the first K tiles need no stage wait: the ring fills while Q is on its way
    for (; k_issued < kStagesK && k_issued < ntile; ++k_issued) issue_tile(k_issued, 0);
  } else if (warp < 4) {
    if (warp == 0) {  // TMEM: two S buffers and O
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_s)),
                   "n"(kTmemCols));
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    // ancestor mask -> registers; without TMA for Q: the Q row -> swizzled shared memory (rows past the tree zero)
    if (row_ok) {
#pragma unroll
      for (int w = 0; w < 4; ++w)
        if (w < p.words) aw[w] = p.anc[((size_t)b * p.Ncap + t_tok) * p.words + w];
    }
    if (!p.q_tma) {
      const __nv_bfloat16* qrow = p.q + (((size_t)b * p.Ncap + t_tok) * p.Hq + h_q) * kHD;
      uint4 qv[16];
#pragma unroll
      for (int c = 0; c < 16; ++c) qv[c] = row_ok ? *reinterpret_cast<const uint4*>(qrow + c * 8) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int c = 0; c < 16; ++c)
        *reinterpret_cast<uint4*>(smem + kSmemQ + (c >> 3) * kRegionQ + swz(r, c & 7)) = qv[c];
      fence_proxy_async();
    }
  }
  // everyone but the producer waits here for the barrier objects, the TMEM address and Q; the producer
  // only signals that the barriers exist (it arrived right after initialising them) and keeps loading
  tc_fence_before();
  if (warp != 4) asm volatile("bar.sync 2, %0;" ::"n"(kThreadsTC) : "memory");
  tc_fence_after();
  // early mode: the softmax warps, the MMA issuer and the spare warp have nothing to do before Q arrives,
  // which is after the wait anyway; the producers wait inside produce()
  if (early && warp != 4 && warp != 6) asm volatile("griddepcontrol.wait;" ::: "memory");
  const uint32_t tmem_base = *tmem_base_s;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + 2 * kBN;

  if (warp == 4) {
    // =========================== TMA producer: K ring ===========================
    produce(0, k_issued, true);  // (this warp has waited, at the latest before the Q load)
  } else if (warp == 6) {
    // =========================== TMA producer: V ring ===========================
    produce(1, 0, !early);
  } else if (warp == 5) {
    // =========================== MMA issuer ===========================
    const uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
    const uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(kHD >> 3) << 17) |
                              ((uint32_t)(kBM >> 4) << 24);  // B operand (V) is MN-major, N = head dim
    // Everything the issue loop computes with is made warp-uniform in the compiler's eyes (a warp reduction
    // of values that are equal in all lanes anyway: the tile count comes from a load, the TMEM address from
    // shared memory), and the ring positions are counters, not remainders: the loop then runs on the uniform
    // datapath, where the MMA instructions take their operands.
    const int ntile_u = __reduce_max_sync(0xffffffffu, ntile);
    const uint32_t tmem_su = __reduce_or_sync(0xffffffffu, tmem_s), tmem_ou = tmem_su + 2 * kBN;
    // descriptors differ only in the start-address field (16-byte units), so they are built once
    const uint64_t dq = umma_desc(smem_u32(smem + kSmemQ), 16, 1024);
    const uint64_t dk = umma_desc(smem_u32(smem + kSmemK), 16, 1024);
    const uint64_t dv = umma_desc(smem_u32(smem + kSmemV), kRegionKV, 1024);
    auto mma_qk = [&](int stage, int buf) {  // S[buf] = Q K^T; releases the K stage (all lanes, converged)
      const uint64_t dks = dk + (uint64_t)(stage * (kTileKV >> 4));
#pragma unroll
      for (int ks = 0; ks < kHD / 16; ++ks)
        umma_bf16(tmem_su + buf * kBN, dq + (uint64_t)((ks >> 2) * (kRegionQ >> 4) + (ks & 3) * 2),
                  dks + (uint64_t)((ks >> 2) * (kRegionKV >> 4) + (ks & 3) * 2), idesc_qk, ks > 0);
      umma_commit(&bar_s[buf]);
      umma_commit(&bar_freek[stage]);
    };
    auto mma_pv = [&](int stage, int buf, bool first) {  // O (+)= P V, P from tensor memory; releases the V stage
      const uint64_t dvs = dv + (uint64_t)(stage * (kTileKV >> 4));
#pragma unroll
      for (int ks = 0; ks < kBN / 16; ++ks)
        umma_bf16_ts(tmem_ou, tmem_su + buf * kBN + ks * 8, dvs + (uint64_t)(ks * (2048 >> 4)), idesc_pv,
                     (!first || ks > 0) ? 1u : 0u);
      umma_commit(&bar_freev[stage]);
    };
    // next scores first: Q K^T of tile it+1 runs while the softmax of tile `it` does; the other CTA on
    // this SM covers the moments when a K tile is late
    bool ok = ntile_u == 0 || ((!p.q_tma || mbar_wait(bar_q, 0)) && mbar_wait(&bar_fullk[0], 0));
    if (ok && ntile_u > 0) {
      tc_fence_after();
      mma_qk(0, 0);
    }
    int ks1 = 1 % kStagesK, kp1 = (1 / kStagesK) & 1;  // K ring position and phase of tile it+1
    int vs0 = 0, vp0 = 0;                              // V ring position and phase of tile it
    for (int it = 0; ok && it < ntile_u; ++it) {
      if (it + 1 < ntile_u) {
        ok = mbar_wait(&bar_fullk[ks1], (uint32_t)kp1);
        if (!ok) break;
        tc_fence_after();
        mma_qk(ks1, (it + 1) & 1);
        if (++ks1 == kStagesK) {
          ks1 = 0;
          kp1 ^= 1;
        }
      }
      ok = mbar_wait(&bar_p[it & 1], (it >> 1) & 1) && mbar_wait(&bar_fullv[vs0], (uint32_t)vp0);
      if (!ok) break;
      tc_fence_after();
      mma_pv(vs0, it & 1, it == 0);
      if (++vs0 == kStagesV) {
        vs0 = 0;
        vp0 ^= 1;
      }
    }
    if (!ok && lane == 0) report(p.st, CAST_ERR_TIMEOUT, b);
  } else if (warp < 4) {
    // =========================== softmax warps ===========================
    // After a wait has expired a thread keeps visiting the barriers (so nobody blocks on it) but
    // touches neither TMEM nor the operand buffers. A warp whose 32 rows all lie past the tree
    // only keeps the barriers in step: its P rows feed output rows nobody reads.
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
    const bool warp_live = row0 + warp * 32 < rows_total;
    const float sc = p.scale_log2;
    float m_used = -INFINITY, l_run = 0.f;  // m_used: the row's reference in raw score units (see below)
    bool ok = true;
    // V rows past the end of the sequence may hold anything (0 * NaN would poison O): zero them (last tile only)
    auto zero_v_tail = [&](int it) {
      const int pos0 = (t0 + it) * kBN, stage = it % kStagesV;
      if (ok && total - pos0 < kBN) {
        ok = mbar_wait(&bar_fullv[stage], (it / kStagesV) & 1);  // the tile has landed
        if (ok) {
          const int valid = total - pos0;
          unsigned char* vbase = smem + kSmemV + stage * kTileKV;
          for (int i = tid; i < (kBN - valid) * 16; i += kSoftmaxThreads) {
            const int rr = valid + (i >> 4), reg = (i >> 3) & 1, c = i & 7;
            *reinterpret_cast<uint4*>(vbase + reg * kRegionKV + rr * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async();  // the MMA reads these rows through the async proxy
        }
      }
    };
    // Every tile takes one pass over its scores: P = 2^(s * scale - m * scale) with a reference m per row that
    // is NOT the running maximum. It starts at 0 and moves, by a whole number of powers of two, only when it has
    // to: when a tile's row sum reaches 2^60 (a score far above the reference; also the case in which the
    // exponential itself overflows, the sum is then inf), or when everything a row has seen so far sums to less
    // than 2^-60 (the reference is far above the scores: their P would drop out of the bottom of the range).
    // Either is rare (scores times scale stay within a few tens of powers of two in a trained model), and in
    // between P is not bounded by 1, which bf16 and the fp32 accumulators have the range for: after every tile a
    // row's sum lies in [2^-60, 2^66], 60 binades from either end. Nothing of a tile is written before its row
    // sums are known, so when a reference has to move the tile's scores are still intact in tensor memory: the
    // new reference is the larger of the tile's largest exponent and that of what is accumulated, both rounded
    // up to a whole power of two; O and the running sum are scaled by 2^-k, which is exact; the tile is evaluated
    // again. (An earlier version took two passes - row maximum, then P - over the first tile of every piece.)
    // Nothing but the scores is awaited: P goes into the score buffer it came from, and that buffer was last
    // read by P V of tile it-2, which the tensor pipe finished before it produced these scores. So the softmax
    // of this tile runs while P V of the previous one does. The second half of a tile's scores is loaded while
    // the first half is computed. (Loading the next tile's first half ahead as well, or handing P over later,
    // was tried in several forms and lost each time.)
    if (!warp_live) {
      // no live rows: stay in step - wait for a tile's scores like the others, so as not to arrive on
      // bar_p[it & 1] before the phase of tile it-2 is over
      for (int it = 0; it < ntile; ++it) {
        if (ok && it >= 1) ok = mbar_wait(&bar_s[it & 1], (it >> 1) & 1);
        zero_v_tail(it);
        tc_fence_before();
        mbar_arrive(&bar_p[it & 1]);
      }
    } else {
      m_used = 0.f;
      const unsigned long long sc2 = pack_f2(sc, sc);
      for (int it = 0; it < ntile; ++it) {
        uint32_t sra[32];
        if (ok) {
          ok = mbar_wait(&bar_s[it & 1], (it >> 1) & 1);
          if (ok) {
            tc_fence_after();
            tmem_ld32(tmem_s + (it & 1) * kBN + lane_sel, sra);
          }
        }
        if (!ok) {  // a wait ran out: keep the barriers in step and nothing else
          tc_fence_before();
          mbar_arrive(&bar_p[it & 1]);
          continue;
        }
        const int buf = it & 1;
        const int pos0 = (t0 + it) * kBN;
        const uint32_t tp = tmem_s + buf * kBN + lane_sel;
        const bool plain = pos0 + kBN <= L;  // wholly inside the prefix: nothing masked (rows past the tree: see neg_ms)
        uint32_t v0 = 0xffffffffu, v1 = 0xffffffffu;  // visibility of this row's 64 columns
        if (!plain) {
          v0 = vis_bits32(aw, pos0 - L);
          v1 = vis_bits32(aw, pos0 - L + 32);
          if (!row_ok) v0 = v1 = 0u;
        }
        // a row past the tree takes -inf: its P is 0 for every finite score, with no masking
        float neg_ms = row_ok ? -m_used * sc : -INFINITY;
        uint32_t pk[2][16];
        unsigned long long lacc = pack_f2(0.f, 0.f);
        {
          const unsigned long long neg2 = pack_f2(neg_ms, neg_ms);
          uint32_t srb[32];
          // Two copies of the arithmetic behind one warp-uniform branch: written as a test inside the loop the
          // masking was compiled into selects that every tile paid for (two instructions per score on
          // top of five per pair), and all tiles but the last one or two are unmasked.
          tmem_wait_ld_regs(sra);
          tmem_ld32(tp + 32, srb);  // in flight while the first half is computed
          if (plain) softmax_half<false>(sra, sc2, neg2, 0u, lacc, pk[0]);
          else softmax_half<true>(sra, sc2, neg2, v0, lacc, pk[0]);
          tmem_wait_ld_regs(srb);
          if (plain) softmax_half<false>(srb, sc2, neg2, 0u, lacc, pk[1]);
          else softmax_half<true>(srb, sc2, neg2, v1, lacc, pk[1]);
        }
        float l0, l1;
        unpack_f2(lacc, l0, l1);
        const bool far = row_ok && !(l0 + l1 < 1.15e18f);  // 2^60
        const bool low = row_ok && (plain || (v0 | v1) != 0u) && (l_run + l0 + l1 < 8.6e-19f);  // 2^-60, something visible
        if (__any_sync(0xffffffffu, far || low)) {
          if (it > 0) ok = mbar_wait(&bar_freev[(it - 1) % kStagesV], ((it - 1) / kStagesV) & 1);  // O must be at rest
          if (ok) {
            tc_fence_after();
            float mxt = -INFINITY;
#pragma unroll 1
            for (int hh = 0; hh < 2; ++hh) {
              uint32_t sr[32];
              tmem_ld32(tp + hh * 32, sr);
              tmem_wait_ld();
              const uint32_t vv = hh ? v1 : v0;
#pragma unroll
              for (int c = 0; c < 32; ++c)  // (`plain ||`: v0 / v1 then stay out of the unmasked path's live registers)
                mxt = fmaxf(mxt, (plain || ((vv >> c) & 1u)) ? __uint_as_float(sr[c]) : -INFINITY);
            }
            float kf = 0.f;
            if (far || low) {
              const float e_tile = mxt > -INFINITY ? fmaf(mxt, sc, neg_ms) : -INFINITY;  // the tile's largest exponent
              const float e_acc = l_run > 0.f ? log2f(l_run) : -INFINITY;                // that of what is accumulated
              const float e = fmaxf(e_tile, e_acc);
              if (e > -INFINITY && e < INFINITY) {
                kf = ceilf(e);
                kf = kf < -1.0e9f ? -1.0e9f : (kf > 1.0e9f ? 1.0e9f : kf);
              }
            }
            // 2^-k for what is accumulated: nothing is (a sum of 0 means every P so far was exactly 0), or its
            // exponent is at most k, so the product cannot overflow; 0 for k beyond the range (it no longer counts)
            const float alpha = l_run > 0.f ? ldexpf(1.f, -(int)kf) : 1.f;
            if (it > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll 1
              for (int q4 = 0; q4 < 4; ++q4) {  // O follows (P V of tile it-1 is over)
                uint32_t orr[32];
                const uint32_t ta = tmem_o + lane_sel + q4 * 32;
                tmem_ld32(ta, orr);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 32; ++c) orr[c] = __float_as_uint(__uint_as_float(orr[c]) * alpha);
                tmem_st32(ta, orr);
              }
            }
            l_run *= alpha;
            neg_ms -= kf;
            m_used += kf / sc;
            l0 = l1 = 0.f;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {  // the tile again (rows that did not move get the same values)
              uint32_t sr[32];
              tmem_ld32(tp + hh * 32, sr);
              tmem_wait_ld();
              const uint32_t vv = plain ? 0xffffffffu : (hh ? v1 : v0);
#pragma unroll
              for (int e = 0; e < 16; ++e) {
                const int c = 2 * e;
                float p0 = fast_exp2(fmaf(__uint_as_float(sr[c]), sc, neg_ms));
                float p1 = fast_exp2(fmaf(__uint_as_float(sr[c + 1]), sc, neg_ms));
                p0 = ((vv >> c) & 1u) ? p0 : 0.f;
                p1 = ((vv >> (c + 1)) & 1u) ? p1 : 0.f;
                l0 += p0;
                l1 += p1;
                const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
                pk[hh][e] = *reinterpret_cast<const uint32_t*>(&pb);
              }
            }
          }
        }
        tmem_st16(tp, pk[0]);
        tmem_st16(tp + 16, pk[1]);
        l_run += l0 + l1;
        tmem_wait_st();
        zero_v_tail(it);
        tc_fence_before();
        mbar_arrive(&bar_p[it & 1]);
      }
    }
    // epilogue: wait for the last P V, then stage O (fp32, unnormalised) and (max, sum) per row in
    // shared memory (the K/V rings, P and Q are idle now): the output rows are written, or merged
    // across the splits, from there in contiguous pieces
    if (ok && ntile > 0) ok = mbar_wait(&bar_freev[(ntile - 1) % kStagesV], ((ntile - 1) / kStagesV) & 1);
    if (!ok) {  // a wait ran out: this split contributes nothing
      m_used = -INFINITY;
      l_run = 0.f;
    }
    if (ok && warp_live && ntile > 0) {
      tc_fence_after();
      if (nsplit > 1) {  // to be merged with other splits: the row normalised by its own sum, in half precision
        const float inv_l = l_run > 0.f ? 1.f / l_run : 0.f;
        __half* sh = reinterpret_cast<__half*>(stage_o) + r * kStageStrideH;
#pragma unroll
        for (int hh = 0; hh < 4; ++hh) {
          uint32_t orr[32];
          tmem_ld32(tmem_o + lane_sel + hh * 32, orr);
          tmem_wait_ld();
#pragma unroll
          for (int c8 = 0; c8 < 4; ++c8) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const __half2 h2 = __floats2half2_rn(__uint_as_float(orr[c8 * 8 + 2 * e]) * inv_l,
                                                   __uint_as_float(orr[c8 * 8 + 2 * e + 1]) * inv_l);
              pk[e] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            *reinterpret_cast<uint4*>(sh + hh * 32 + c8 * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
      } else {
#pragma unroll
        for (int hh = 0; hh < 4; ++hh) {
          uint32_t orr[32];
          tmem_ld32(tmem_o + lane_sel + hh * 32, orr);
          tmem_wait_ld();
          float* so = stage_o + r * kStageStride + hh * 32;
#pragma unroll
          for (int c4 = 0; c4 < 8; ++c4)
            *reinterpret_cast<float4*>(so + c4 * 4) =
                make_float4(__uint_as_float(orr[c4 * 4]), __uint_as_float(orr[c4 * 4 + 1]), __uint_as_float(orr[c4 * 4 + 2]),
                            __uint_as_float(orr[c4 * 4 + 3]));
        }
      }
    }
    stage_ml[r * 2] = l_run > 0.f ? m_used * sc * 0.69314718055994531f : -INFINITY;  // natural-log units (-inf: nothing visible)
    stage_ml[r * 2 + 1] = l_run;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {  // every TMEM access of this CTA is over
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols));
  }
  if (cs > 1) cluster_sync_all();  // every CTA of the cluster has staged its rows
  const int rows_here = rows_total - row0 < kBM ? rows_total - row0 : kBM;
  if (nsplit == 1) {
    for (int rr = warp; rr < rows_here; rr += kThreadsTC / 32) {
      const int grow = grow0 + rr, tt = grow / G, hh = kvh * G + grow % G;
      const float4 o4 = *reinterpret_cast<const float4*>(stage_o + rr * kStageStride + lane * 4);
      const float l_tot = stage_ml[rr * 2 + 1];
      const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
      const __nv_bfloat162 a = __floats2bfloat162_rn(o4.x * inv, o4.y * inv), c2 = __floats2bfloat162_rn(o4.z * inv, o4.w * inv);
      uint2 pk;
      pk.x = *reinterpret_cast<const uint32_t*>(&a);
      pk.y = *reinterpret_cast<const uint32_t*>(&c2);
      *reinterpret_cast<uint2*>(p.out + (((size_t)b * p.Ncap + tt) * p.Hq + hh) * kHD + lane * 4) = pk;
    }
  } else if (cs == 0) {
    // global-merge mode: partials to the workspace; the last split of this row block to finish merges
    const __half* sh = reinterpret_cast<const __half*>(stage_o);
    for (int rr = warp; rr < rows_here; rr += kThreadsTC / 32) {
      const int grow = grow0 + rr, tt = grow / G, hh = kvh * G + grow % G;
      const size_t pr = (((size_t)b * p.Hq + hh) * p.Ncap + tt) * p.nsplit_max + split;
      __stcg(reinterpret_cast<uint2*>(p.part_o + pr * kHD + lane * 4),
             *reinterpret_cast<const uint2*>(sh + rr * kStageStrideH + lane * 4));
      if (lane == 0) {
        __stcg(p.part_ml + pr * 2, stage_ml[rr * 2]);
        __stcg(p.part_ml + pr * 2 + 1, stage_ml[rr * 2 + 1]);
      }
    }
    __syncthreads();
    if (tid == 0) {
      // one acquire-release atomic at device scope: releases this CTA's partials (the barrier above made
      // them this thread's to release), acquires those of the splits that finished earlier
      int32_t* cnt = p.ticket + ((size_t)b * p.Hkv + kvh) * p.nrb + rb;
      int t;
      asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(t) : "l"(cnt) : "memory");
      *last_s = (t == nsplit - 1);
      if (t == nsplit - 1) *cnt = 0;  // ready for the next launch
    }
    __syncthreads();
    if (*last_s) {
      if (nsplit <= 2) merge_rows_global<4, 2>(p, b, kvh, grow0, rows_here, nsplit);
      else if (nsplit <= 4) merge_rows_global<4, 4>(p, b, kvh, grow0, rows_here, nsplit);
      else merge_rows_global<2, kMaxSplit>(p, b, kvh, grow0, rows_here, nsplit);
    }
  } else {
    const uint32_t so_s = smem_u32(stage_o), sml_s = smem_u32(stage_ml);
    const int rank0 = crank - split;  // first CTA of this row block's split group
    if (nsplit <= 2) merge_rows<8, 2>(p, so_s, sml_s, rank0, b, kvh, grow0, rows_here, nsplit, split);
    else if (nsplit <= 4) merge_rows<4, 4>(p, so_s, sml_s, rank0, b, kvh, grow0, rows_here, nsplit, split);
    else merge_rows<2, kMaxSplit>(p, so_s, sml_s, rank0, b, kvh, grow0, rows_here, nsplit, split);
  }
  if (cs > 1) cluster_sync_all();  // nobody leaves while a peer may still read its shared memory
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

// Q [B * Ncap tokens][Hq heads][128 dims]: a box is 128 / G tokens x G heads x 64 dims (one row block, one half)
bool make_q_map(CUtensorMap* map, const void* base, int B, int Ncap, int Hq, int G) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  const cuuint64_t dims[3] = {kHD, (cuuint64_t)Hq, (cuuint64_t)B * Ncap};
  const cuuint64_t strides[2] = {kHD * 2, (cuuint64_t)Hq * kHD * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)(kBM / G)};
  const cuuint32_t estr[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
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

// What the host decides for one launch shape: the launch mode, the grid and the workspace it needs.
struct TcPlan {
  int nrb, splits, rpc, cs, nsplit_max;
  bool cluster_mode;
  long long grid;
  size_t ws_bytes, rows;  // global-merge mode: workspace size and partial rows (0: none)
};
constexpr size_t kTicketBytes = (size_t)CAST_MAX_BATCH * 256 * sizeof(int32_t);

bool tc_shape_ok(int D, int page_size) {
  if (D != kHD) return false;
  return page_size == 0 || (page_size >= 8 && page_size <= kBN && (kBN % page_size) == 0 && (page_size % 8) == 0);
}

bool tc_plan(const cast_ctx* c, int B, int Hq, int Hkv, int page_size, int seq_capacity, TcPlan* pl) {
  const int G = Hq / Hkv, Ncap = c->cfg.max_tree;
  // no tree of this context has more than total_token nodes: row blocks past that are never launched
  const int Nmax = c->cfg.total_token < Ncap ? c->cfg.total_token : Ncap;
  const int nrb = (Nmax * G + kBM - 1) / kBM;
  const int max_pos = page_size == 0 ? seq_capacity : seq_capacity * page_size;
  const int max_tiles = (max_pos + kBN - 1) / kBN;
  // KV splits per row block: as many (a power of two, at most 8) as keep the CTA count within one
  // wave of two CTAs per SM, and no more than leave each split a few tiles. The tree sizes are only
  // known on the device, so this is sized for the largest tree; a cluster then covers `rpc` row blocks
  // and hands the CTAs of absent ones to the present ones as further splits.
  const int slots = 2 * c->num_sms;
  int splits = 1;
  while (splits < kMaxSplit && (long long)B * Hkv * nrb * splits * 2 <= slots && max_tiles / (splits * 2) >= 2) splits *= 2;
  int rpc = 1;
  while (rpc * 2 * splits <= kMaxSplit && rpc * 2 <= nrb) rpc *= 2;
  // Clusters pay when CTAs are short (the merge through distributed shared memory is cheap and the
  // splits are what fills the machine). With long CTAs, or so many sequences that nothing needs
  // splitting on average, an even load matters more: no clusters, pieces sized on the device.
  // (with B * Hkv items or more than the machine has slots, nothing is ever split: plain launch, cs = 1)
  const bool cluster_mode = (splits > 1 && max_tiles / splits <= 64) || (long long)B * Hkv >= slots;
  if ((long long)B * Hkv >= slots) splits = rpc = 1;
  pl->nrb = nrb; pl->splits = splits; pl->rpc = rpc; pl->cluster_mode = cluster_mode;
  pl->ws_bytes = 0; pl->rows = 0;
  if (cluster_mode) {
    pl->cs = splits * rpc;
    const int groups = (nrb + rpc - 1) / rpc;
    pl->grid = (long long)B * Hkv * groups * pl->cs;
    pl->nsplit_max = 1;
  } else {
    pl->cs = 1;
    int nsplit_max = kMaxSplit < max_tiles ? kMaxSplit : max_tiles;
    if (nsplit_max < 1) nsplit_max = 1;
    const long long waves = ((long long)B * Hkv * nrb + slots - 1) / slots;
    pl->grid = (long long)slots * (waves < 1 ? 1 : waves);
    pl->nsplit_max = nsplit_max;
    if (nsplit_max > 1) {
      // workspace: a fixed ticket region (B * Hkv * nrb <= 64 * Hq entries), then the partials
      if ((size_t)B * Hkv * nrb * sizeof(int32_t) > kTicketBytes) return false;
      pl->rows = (size_t)B * Hq * Ncap * nsplit_max;
      pl->ws_bytes = kTicketBytes + pl->rows * (kHD * sizeof(__half) + 2 * sizeof(float));
    }
  }
  return pl->grid <= 0x7fffffffll;
}

}  // namespace

// Workspace bytes a tensor-core launch of this shape needs (0: none, or the shape is not the tensor path's).
size_t tree_attention_tc_workspace(const cast_ctx* c, int B, int Hq, int Hkv, int D, int page_size, int seq_capacity) {
  TcPlan pl;
  if (!tc_shape_ok(D, page_size) || !tc_plan(c, B, Hq, Hkv, page_size, seq_capacity, &pl)) return 0;
  return pl.ws_bytes;
}
// Grows the tensor path's workspace to `bytes` (set-up time only: synchronises and allocates).
cast_status tree_attention_tc_reserve(cast_ctx* c, size_t bytes) {
  if (bytes <= c->attn_tc_ws_bytes) return CAST_OK;
  CAST_CUDA_OK(cudaDeviceSynchronize());
  if (c->attn_tc_ws) cudaFree(c->attn_tc_ws);
  c->attn_tc_ws = nullptr;
  c->attn_tc_ws_bytes = 0;
  CAST_CUDA_OK(cudaMalloc(&c->attn_tc_ws, bytes));
  // tickets start at zero; every merge leaves its ticket at zero again
  CAST_CUDA_OK(cudaMemset(c->attn_tc_ws, 0, kTicketBytes));
  c->attn_tc_ws_bytes = bytes;
  return CAST_OK;
}

bool tree_attention_tc_launch(cast_ctx* c, const void* q, const void* k, const void* v, int B, int Hq, int Hkv, int D,
                              int page_size, const int32_t* page_table, int seq_capacity, int num_pages,
                              const int32_t* kv_len, const uint32_t* anc, const int32_t* n_tree, const int32_t* first_row,
                              float scale, void* out, cudaStream_t stream, cast_status* status) {
  if (!tc_shape_ok(D, page_size) || !(scale > 0.f)) return false;
  if ((((uintptr_t)k | (uintptr_t)v) & 127) != 0) return false;
  TcPlan pl;
  if (!tc_plan(c, B, Hq, Hkv, page_size, seq_capacity, &pl)) return false;
  CUtensorMap map_k, map_v;
  if (!make_kv_map(&map_k, k, B, Hkv, page_size, seq_capacity, num_pages) ||
      !make_kv_map(&map_v, v, B, Hkv, page_size, seq_capacity, num_pages))
    return false;
  const int G = Hq / Hkv, Ncap = c->cfg.max_tree;
  const int Nmax = c->cfg.total_token < Ncap ? c->cfg.total_token : Ncap;
  CUtensorMap map_q = map_k;  // (a valid descriptor either way; used only when q_tma is set)
  const bool q_tma = G <= kBM && (kBM % G) == 0 && make_q_map(&map_q, q, B, Ncap, Hq, G);
  TcParams p;
  p.q_tma = q_tma ? 1 : 0;
  p.early = (c->attn_early && !c->tree_inputs_fresh && q_tma) ? 1 : 0;
  p.q = (const __nv_bfloat16*)q; p.out = (__nv_bfloat16*)out;
  p.B = B; p.Ncap = Ncap; p.Nmax = Nmax; p.Hq = Hq; p.Hkv = Hkv; p.G = G; p.page_size = page_size;
  p.seq_capacity = seq_capacity; p.num_pages = num_pages; p.words = c->words;
  p.page_table = page_table; p.kv_len = kv_len; p.n_tree = n_tree; p.first_row = first_row; p.anc = anc;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.st = c->state;
  p.num_sms = c->num_sms; p.nrb = pl.nrb;
  p.part_o = nullptr; p.part_ml = nullptr; p.ticket = nullptr;
  *status = CAST_OK;
  const long long grid = pl.grid;
  const int cs = pl.cs;
  p.rpc = pl.rpc; p.nsplit_max = pl.nsplit_max;
  p.cs = pl.cluster_mode ? cs : 0;
  if (pl.ws_bytes > 0) {
    // compute calls never allocate: the workspace comes from cast_reserve_attention
    if (pl.ws_bytes > c->attn_tc_ws_bytes) {
      *status = CAST_ERR_CAPACITY;
      return true;
    }
    p.ticket = reinterpret_cast<int32_t*>(c->attn_tc_ws);
    p.part_o = reinterpret_cast<__half*>(reinterpret_cast<char*>(c->attn_tc_ws) + kTicketBytes);
    p.part_ml = reinterpret_cast<float*>(p.part_o + pl.rows * kHD);
  }
  // The work list: under the caller's promise the lengths and tree sizes do not change between the attention
  // calls of a step, so what every CTA would decode for itself is decoded once, by a small kernel launched in
  // front of the first such call (or when the call's shape changes), and the calls after it read one item each.
  p.worklist = nullptr;
  if (c->attn_early && first_row == nullptr && grid <= kAttnWorkListCap) {  // (a window call names new sizes every time)
    const unsigned long long key[8] = {(unsigned long long)(uintptr_t)n_tree, (unsigned long long)(uintptr_t)kv_len,
                                       (unsigned long long)(uintptr_t)first_row,
                                       ((unsigned long long)B << 48) | ((unsigned long long)Hq << 32) | ((unsigned long long)Hkv << 16) | (unsigned)page_size,
                                       ((unsigned long long)seq_capacity << 32) | (unsigned)grid,
                                       ((unsigned long long)(unsigned)p.cs << 32) | ((unsigned)p.rpc << 16) | (unsigned)p.nsplit_max,
                                       (unsigned long long)Nmax, (unsigned long long)c->num_sms};
    bool same = c->wl_valid && !c->tree_inputs_fresh;
    for (int i = 0; i < 8 && same; ++i) same = c->wl_key[i] == key[i];
    if (!same) {
      attn_worklist_kernel<<<(unsigned)((grid + 7) / 8), 256, 0, stream>>>(p, (int)grid, c->attn_worklist);
      if (cudaGetLastError() != cudaSuccess) { *status = CAST_ERR_CUDA; return true; }
      for (int i = 0; i < 8; ++i) c->wl_key[i] = key[i];
      c->wl_valid = 1;
      p.early = 0;  // the list is the previous kernel's: read it after the wait
    }
    p.worklist = c->attn_worklist;
  }
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(tree_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) !=
        cudaSuccess) {
      *status = CAST_ERR_CUDA;
      return true;
    }
    // two CTAs per SM need the largest shared-memory carve-out
    cudaFuncSetAttribute(tree_attn_tc_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    attr_done = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3(kThreadsTC, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // may become resident before the previous kernel of the stream has drained (the kernel waits where it must)
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel, p, map_k, map_v, map_q) != cudaSuccess) {
    cudaGetLastError();
    *status = CAST_ERR_CUDA;
    return true;
  }
  *status = launch_status();
  return true;
}

}  // namespace cast
