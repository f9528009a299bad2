// Projection and back-projection of the GaLore step on the 5th-generation
// tensor cores (sm_100a): bf16 operands staged in shared memory by TMA,
// tcgen05.mma with fp32 accumulators in tensor memory, epilogues that either
// store split-K partial sums of R or apply the update to W in place
// (Algorithm 1: R = P^T G resp. G Q;  W <- W - lr * alpha * P N resp. N Q^T).
//
// With one K slice per output tile the projection's epilogue also runs Adam on its tile of R
// (moment update, bias correction, Eq. 15, 8-bit dequantisation and requantisation of the moments)
// and writes the normalised update N for the back-projection: R never reaches memory.
//
// One persistent CTA per SM:
//   warp 0        TMA producer: fills a ring of kStages shared-memory stages
//   warp 1        MMA issuer (one lane) and owner of the tensor-memory allocation
//   warps 2..     epilogue (four warps, eight when it runs Adam): tcgen05.ld of a finished
//                 accumulator, then global memory
// Two accumulators of kBN columns alternate, so the epilogue of one tile runs
// under the MMAs of the next.  Work units are (tile_m, tile_n, K slice); the
// K slices of one output tile go to separate partial buffers that the Adam
// kernel sums in a fixed order, so results do not depend on scheduling.
//
// Every wait on an mbarrier is bounded by a clock limit; when it runs out the
// CTA latches GALORE_DEV_WAIT_EXPIRED, lets its outstanding copies land,
// releases tensor memory and returns.
#include "gemm_tc.cuh"

#include <cudaTypedefs.h>

#include "adam.cuh"

#include <algorithm>
#include <memory>
#include <mutex>
#include <new>

namespace galore {

namespace {

constexpr int kBM = 128;          // rows of an output tile = TMEM lanes
constexpr int kBN = 256;          // columns of an output tile = TMEM columns per accumulator
constexpr int kBK = 64;           // K per stage: 64 bf16 = one 128-byte swizzle row
constexpr int kUmmaK = 16;
constexpr uint32_t kTmemCols = 512;
constexpr int kABytes = kBM * kBK * 2;            // 16 KiB: the 128 rows of A one CTA stages per k-block

// CTAS = 1: one CTA computes a 128 x 256 tile.  CTAS = 2: a cluster of two CTAs computes 256 x 256
// with cta_group::2 MMAs; each CTA stages its own 128 rows of A and half (128 columns) of B, so a
// k-block costs 32 KiB of shared-memory fill per CTA instead of 48 and the ring holds 6 stages.
template <int CTAS>
struct Geo {
  static constexpr int kTileM = kBM * CTAS;
  static constexpr int kBNcta = kBN / CTAS;
  static constexpr int kBBytes = kBNcta * kBK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStages = CTAS == 1 ? 4 : 6;
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /* alignment slack */ + 256 /* barriers */;
};
constexpr long long kWaitLimitCycles = 4000000000LL;   // about two seconds

// EPI_APPLY_DECAY is EPI_APPLY with W multiplied by TcParams::keep first (GaLore-AdamW).  It is an
// instantiation of its own: the same code with the multiply behind a run-time test made the plain
// update 15 % slower at K = 512.
// EPI_ADAM_F32 / EPI_ADAM_Q8: the projection with Adam on its output tile (fp32 / 8-bit moments).
enum { EPI_PARTIAL = 0, EPI_APPLY = 1, EPI_APPLY_DECAY = 2, EPI_ADAM_F32 = 3, EPI_ADAM_Q8 = 4 };
constexpr bool epi_is_adam(int epi) { return epi == EPI_ADAM_F32 || epi == EPI_ADAM_Q8; }
// Adam is instruction-heavy (about 70 per element with 8-bit moments) and every element is a chain
// of dependent lookups and arithmetic: sixteen epilogue warps, four per quarter of the accumulator's
// lanes with 64 columns each, give every scheduler of the SM four warps to switch between while the
// tensor cores work on the next tile (eight warps of 128 columns each ran three times longer than
// the MMAs of a tile).
constexpr int epi_warps(int epi) { return epi_is_adam(epi) ? 16 : 4; }
constexpr int epi_threads(int epi) { return 64 + 32 * epi_warps(epi); }     // + producer warp and MMA warp
constexpr int epi_smem(int epi) { return epi == EPI_ADAM_Q8 ? (int)sizeof(Q8Tables) : 0; }

constexpr int kMaxGroup = 32;     // problems one launch can carry (its arguments travel as kernel parameters)

struct TcParams {
  int M, N, K;
  int tile_m;                 // rows of a work unit: 128 (one CTA) or 256 (CTA pair)
  int a_mn, b_mn;             // operand majors in shared memory: 1 = M/N contiguous, 0 = K contiguous
  int tiles_m, tiles_n, splits;
  int kblocks_total, kblocks_per_split;
  int m_fast;                 // 1: consecutive units walk tile_m first (B panel shared), 0: tile_n first
  // EPI_PARTIAL
  float* part;
  int64_t ld_part, split_stride;
  // EPI_APPLY
  void* W;
  int64_t ldw;
  int vec32;                  // W base and row pitch (resp. the partial buffer's) are 32-byte aligned
  float scale;
  float keep;                 // EPI_APPLY_DECAY: W is multiplied by this before the update is subtracted
  int32_t* status;
  // EPI_ADAM_*: the state of the layer (rows x cols of the output, row pitch ld_s) and where N goes
  float *Ms, *Vs;             // fp32 moments, or
  uint8_t *Mc, *Vc;           // 8-bit codes with
  float *Mam, *Vam;           // one absmax per tile of q_rows x 64 state elements, tile (I, J) at I * q_tiles_c + J
  int64_t ld_s;
  int q_rows, q_tiles_c;
  __nv_bfloat16* Nout;
  int64_t ld_n;
  int adam_vec;               // bases and pitches of the state and of N allow 32-byte accesses
  AdamParams ap;
};

// One launch = up to kMaxGroup independent problems; work units are numbered across them.
struct TcGroup {
  CUtensorMap map_a[kMaxGroup];
  CUtensorMap map_b[kMaxGroup];
  TcParams p[kMaxGroup];
  int unit_end[kMaxGroup];    // running total of units: problem i owns [unit_end[i-1], unit_end[i])
  int count;
  Q8TablePtrs q8;             // EPI_ADAM_Q8: the code tables in global memory
};

// ---- PTX wrappers ---------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false when the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitLimitCycles) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

// ---- CTA pairs ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load of a CTA pair: data lands in this CTA, completion is signalled on the leader's barrier
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t leader_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(leader_bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_result, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D (+)= A B over the pair: 256 x kBN x 16; A rows and B columns are split between the two CTAs
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// one arrival on the barrier at this offset in both CTAs once the pair's MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], 128 x kBN x 16, bf16 in, fp32 out
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// the mbarrier receives one arrival once every MMA issued so far by this thread has finished
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread t of the warp gets lane (base lane + t)
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// 32-byte global accesses: one request covers a whole 32-byte sector, so a thread that walks its own
// row does not send half-filled sectors through the L1/L2 fabric.  Address must be 32-byte aligned.
__device__ __forceinline__ void ld_global_32B(const void* ptr, uint4& a, uint4& b) {
  asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w)
               : "l"(ptr)
               : "memory");
}
__device__ __forceinline__ void st_global_32B(void* ptr, const uint4& a, const uint4& b) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               ::"l"(ptr), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w)
               : "memory");
}

// ---- descriptors ------------------------------------------------------------------------
// Shared-memory operand descriptor, 128-byte swizzle, tile base 1024-byte aligned.
//  K-major  : rows of 64 bf16 (128 B); 8-row groups 1024 B apart (stride offset); leading offset unused.
//  MN-major : 64-element (128 B) runs along M/N, one per k; 8-k groups 1024 B apart (stride offset);
//             the next 64 elements of M/N start kBK * 128 B further on (leading offset).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, bool mn_major) {
  const uint64_t lbo = mn_major ? (uint64_t)((kBK * 128) >> 4) : 1ull;
  const uint64_t sbo = 1024 >> 4;
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | (lbo << 16) | (sbo << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor: fp32 accumulate, bf16 x bf16, majors, N, M.
__host__ __device__ constexpr uint32_t instr_desc(int a_mn, int b_mn, int tile_m) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(tile_m >> 4) << 24);
}

struct Unit {
  int m0, n0, split, kb_begin, kb_end;
};

__device__ __forceinline__ Unit decode_unit(const TcGroup& g, int u, int& pi) {
  pi = 0;
  while (pi + 1 < g.count && u >= g.unit_end[pi]) ++pi;
  if (pi > 0) u -= g.unit_end[pi - 1];
  const TcParams& p = g.p[pi];
  int tm, tn, s;
  if (p.m_fast) {
    tm = u % p.tiles_m;
    s = (u / p.tiles_m) % p.splits;
    tn = u / (p.tiles_m * p.splits);
  } else {
    tn = u % p.tiles_n;
    s = (u / p.tiles_n) % p.splits;
    tm = u / (p.tiles_n * p.splits);
  }
  Unit w;
  w.m0 = tm * p.tile_m;
  w.n0 = tn * kBN;
  w.split = s;
  w.kb_begin = s * p.kblocks_per_split;
  w.kb_end = min(p.kblocks_total, w.kb_begin + p.kblocks_per_split);
  return w;
}

// ---- epilogues ----------------------------------------------------------------------------

// thread owns row `row`, columns [col0, col0 + 32) of the tile
__device__ __forceinline__ void epi_partial(const TcParams& p, const Unit& w, int row, int col0, const uint32_t (&v)[32]) {
  if (row >= p.M) return;
  float* dst = p.part + (int64_t)w.split * p.split_stride + (int64_t)row * p.ld_part + col0;
  if (col0 + 32 <= p.N && p.vec32) {
#pragma unroll
    for (int j = 0; j < 32; j += 8)
      st_global_32B(dst + j, make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]), make_uint4(v[j + 4], v[j + 5], v[j + 6], v[j + 7]));
  } else if (col0 + 32 <= p.N && (p.ld_part & 3) == 0) {
#pragma unroll
    for (int j = 0; j < 32; j += 4)
      *reinterpret_cast<float4*>(dst + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                        __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
  } else {
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (col0 + j < p.N) dst[j] = __uint_as_float(v[j]);
  }
}

// w <- w - scale * acc, or keep * w - scale * acc (decoupled weight decay)
template <bool DECAY>
__device__ __forceinline__ float apply_one(float w, float acc, float scale, float keep) {
  return DECAY ? fmaf(-scale, acc, keep * w) : fmaf(-scale, acc, w);
}

// one 16-byte vector of W
template <typename TW, bool DECAY>
__device__ __forceinline__ void apply_vec(uint4& raw, const uint32_t* acc, float scale, float keep) {
  if constexpr (sizeof(TW) == 2) {
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float2 f = __bfloat1622float2(h[q]);
      f.x = apply_one<DECAY>(f.x, __uint_as_float(acc[2 * q]), scale, keep);
      f.y = apply_one<DECAY>(f.y, __uint_as_float(acc[2 * q + 1]), scale, keep);
      h[q] = __floats2bfloat162_rn(f.x, f.y);
    }
  } else {
    float4* f = reinterpret_cast<float4*>(&raw);
    f->x = apply_one<DECAY>(f->x, __uint_as_float(acc[0]), scale, keep);
    f->y = apply_one<DECAY>(f->y, __uint_as_float(acc[1]), scale, keep);
    f->z = apply_one<DECAY>(f->z, __uint_as_float(acc[2]), scale, keep);
    f->w = apply_one<DECAY>(f->w, __uint_as_float(acc[3]), scale, keep);
  }
}

// edge tiles: thread owns row `row`, columns [col0, col0 + 32) of the tile
template <typename TW, bool DECAY>
__device__ __forceinline__ void epi_apply(const TcParams& p, int row, int col0, const uint32_t (&v)[32]) {
  if (row >= p.M) return;
  TW* dst = (TW*)p.W + (int64_t)row * p.ldw + col0;
  constexpr int kVec = 16 / (int)sizeof(TW);
  if (col0 + 32 <= p.N) {
#pragma unroll
    for (int j = 0; j < 32; j += kVec) {
      uint4 raw = *reinterpret_cast<const uint4*>(dst + j);
      apply_vec<TW, DECAY>(raw, &v[j], p.scale, p.keep);
      *reinterpret_cast<uint4*>(dst + j) = raw;
    }
  } else {
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (col0 + j < p.N) dst[j] = cvt<TW>(apply_one<DECAY>(cvt<float>(dst[j]), __uint_as_float(v[j]), p.scale, p.keep));
  }
}


// ---- Adam in the projection's epilogue ----------------------------------------------------------
// The thread owns row `row` of R and the kAdamCols columns from col0 on (Algorithm 1, the update
// block on its part of R; Eq. 15 for N), and walks them kAdamChunk at a time.  Rows and columns
// outside the matrix hold exact zeros in the accumulator (TMA fills out-of-range operand elements
// with zeros).
constexpr int kAdamCols = kStateTileCols;    // 64: columns per epilogue warp = width of a quantisation block
constexpr int kAdamChunk = 16;

// 32 lanes x 16 consecutive fp32 columns
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}

// 16 values of N as bf16: one 32-byte store when the row allows it
__device__ __forceinline__ void st_n16(__nv_bfloat16* dst, const float (&n)[16], bool vec, int valid) {
  if (vec) {
    uint32_t w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(n[2 * j], n[2 * j + 1]);
      w[j] = *reinterpret_cast<const uint32_t*>(&h);
    }
    st_global_32B(dst, make_uint4(w[0], w[1], w[2], w[3]), make_uint4(w[4], w[5], w[6], w[7]));
  } else {
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (j < valid) dst[j] = __float2bfloat16_rn(n[j]);
  }
}

__device__ __forceinline__ void ld16f(const float* src, float (&x)[16]) {
#pragma unroll
  for (int j = 0; j < 16; j += 8) {
    uint4 a, b;
    ld_global_32B(src + j, a, b);
    x[j] = __uint_as_float(a.x); x[j + 1] = __uint_as_float(a.y); x[j + 2] = __uint_as_float(a.z); x[j + 3] = __uint_as_float(a.w);
    x[j + 4] = __uint_as_float(b.x); x[j + 5] = __uint_as_float(b.y); x[j + 6] = __uint_as_float(b.z); x[j + 7] = __uint_as_float(b.w);
  }
}
__device__ __forceinline__ void st16f(float* dst, const float (&x)[16]) {
#pragma unroll
  for (int j = 0; j < 16; j += 8)
    st_global_32B(dst + j, make_uint4(__float_as_uint(x[j]), __float_as_uint(x[j + 1]), __float_as_uint(x[j + 2]), __float_as_uint(x[j + 3])),
                  make_uint4(__float_as_uint(x[j + 4]), __float_as_uint(x[j + 5]), __float_as_uint(x[j + 6]), __float_as_uint(x[j + 7])));
}

// fp32 moments: one pass
__device__ __forceinline__ bool epi_adam_f32(const TcParams& p, int row, int col0, uint32_t t_addr, uint32_t accf,
                                             uint32_t acc_phase, volatile int* abort_flag, bool& ok) {
  const bool row_ok = row < p.M;
  const int ncols = row_ok ? max(0, min(kAdamCols, p.N - col0)) : 0;       // columns of this thread inside the matrix
  const bool vec = p.adam_vec != 0;
  const AdamParams ap = p.ap;
  const int64_t so = (int64_t)row * p.ld_s + col0;
  float* __restrict__ Mrow = p.Ms + so;
  float* __restrict__ Vrow = p.Vs + so;
  __nv_bfloat16* __restrict__ Nrow = p.Nout + (int64_t)row * p.ld_n + col0;
  float m[kAdamChunk], v[kAdamChunk];
  auto fetch = [&](int c) {
    const int valid = ncols - c;
    if (valid >= kAdamChunk && vec) {
      ld16f(Mrow + c, m);
      ld16f(Vrow + c, v);
    } else {
#pragma unroll
      for (int j = 0; j < kAdamChunk; ++j) {
        m[j] = j < valid ? Mrow[c + j] : 0.f;
        v[j] = j < valid ? Vrow[c + j] : 0.f;
      }
    }
  };
  fetch(0);                                   // does not depend on the MMAs: in flight while the tile is computed
  // the decision is taken by the warp as a whole: what follows is warp-synchronous
  if (!__all_sync(0xffffffffu, mbar_wait(accf, acc_phase, abort_flag))) { ok = false; return false; }
  tc_fence_after();
  uint32_t top = 0u;      // largest bit pattern among the new second moments (all >= 0): a non-finite r shows here
#pragma unroll 1
  for (int c = 0; c < kAdamCols; c += kAdamChunk) {
    const int valid = ncols - c;
    if (!__any_sync(0xffffffffu, valid > 0)) break;      // the whole warp is past the last column
    if (c > 0) fetch(c);
    uint32_t acc[kAdamChunk];
    tmem_ld_32x16(t_addr + (uint32_t)c, acc);
    tmem_ld_wait();
    float n[kAdamChunk];
#pragma unroll
    for (int j = 0; j < kAdamChunk; ++j) {
      const float r = __uint_as_float(acc[j]);
      m[j] = adam_m(m[j], r, ap);
      v[j] = adam_v(v[j], r, ap);
      n[j] = adam_normalised(m[j], v[j], ap);
      top = max(top, __float_as_uint(v[j]));
    }
    if (valid >= kAdamChunk && vec) {
      st16f(Mrow + c, m);
      st16f(Vrow + c, v);
    } else {
#pragma unroll
      for (int j = 0; j < kAdamChunk; ++j)
        if (j < valid) {
          Mrow[c + j] = m[j];
          Vrow[c + j] = v[j];
        }
    }
    st_n16(Nrow + c, n, valid >= kAdamChunk && vec, valid);
  }
  return top >= 0x7f800000u;
}

// 32 lanes x 8 consecutive fp32 columns
__device__ __forceinline__ void tmem_ld_32x8(uint32_t taddr, uint32_t (&v)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// eight old codes of one moment, columns [c, c + 8) of the thread's stretch: one 8-byte load, or byte by
// byte with the code of zero outside the matrix
__device__ __forceinline__ uint2 ld_codes8(const uint8_t* row, int c, int ncols, bool vec, uint32_t zero_code) {
  if (vec) return *reinterpret_cast<const uint2*>(row + c);
  uint32_t w[2] = {0u, 0u};
#pragma unroll
  for (int k = 0; k < 8; ++k) w[k >> 2] |= (c + k < ncols ? (uint32_t)row[c + k] : zero_code) << (8 * (k & 3));
  return make_uint2(w[0], w[1]);
}

// 8-bit moments.  A quantisation block is a tile of q_rows x 64 state elements: q_rows lanes of this
// warp hold all of it, so its absmax is a warp-shuffle reduction.  Two passes over the accumulator:
// the first finds the block's absmax of the updated moments, the second recomputes them (the same
// instructions, hence the same bits), writes N and the new codes.  Both walk the thread's 64
// columns eight at a time in loops that are NOT unrolled: sixteen warps at different points of a
// fully unrolled body (about 5000 instructions) spent most of their time waiting for instruction
// fetch, and the old codes kept in registers across both passes spilled.  The codes are read once
// per pass instead, the second time from L2.
__device__ __forceinline__ bool epi_adam_q8(const TcParams& p, int row, int col0, uint32_t t_addr, uint32_t accf,
                                            uint32_t acc_phase, volatile int* abort_flag, const Q8Tables& t, bool& ok) {
  constexpr int CH = 8;
  const bool row_ok = row < p.M;
  const int ncols = row_ok ? max(0, min(kAdamCols, p.N - col0)) : 0;
  const bool vec = p.adam_vec != 0 && ncols == kAdamCols;
  const AdamParams ap = p.ap;
  const int64_t so = (int64_t)row * p.ld_s + col0;
  uint8_t* __restrict__ Mrow = p.Mc + so;
  uint8_t* __restrict__ Vrow = p.Vc + so;
  __nv_bfloat16* __restrict__ Nrow = p.Nout + (int64_t)row * p.ld_n + col0;
  const int tile = ncols > 0 ? (row / p.q_rows) * p.q_tiles_c + col0 / kAdamCols : 0;
  // the old codes and the block's old absmax do not depend on the MMAs: asked for now, they arrive
  // while the tile is computed
  if (ncols > 0) {
    prefetch_l2(Mrow);
    prefetch_l2(Vrow);
  }
  const float am_m = ncols > 0 ? p.Mam[tile] : 0.f, am_v = ncols > 0 ? p.Vam[tile] : 0.f;
  // the decision is taken by the warp as a whole: what follows is warp-synchronous
  if (!__all_sync(0xffffffffu, mbar_wait(accf, acc_phase, abort_flag))) { ok = false; return false; }
  tc_fence_after();
  const int wcols = __reduce_max_sync(0xffffffffu, ncols);       // columns any lane of the warp has
  if (wcols == 0) return false;                                  // the warp's part of the tile lies outside the matrix

  // Both passes are software-pipelined by one chunk: the next chunk's accumulator columns and old
  // codes are asked for before the current chunk's arithmetic, which is a chain of dependent
  // shared-memory lookups per element.
  // ---- pass 1: absmax of the updated moments over the block
  float mx_m = 0.f;
  uint32_t mx_vb = 0u;          // v >= 0: bit order is value order; a NaN or an infinity ends up on top
  {
    uint2 nm = ld_codes8(Mrow, 0, ncols, vec, 127u), nv = ld_codes8(Vrow, 0, ncols, vec, 0u);
    uint32_t nacc[CH];
    tmem_ld_32x8(t_addr, nacc);
#pragma unroll 1
    for (int c = 0; c < wcols; c += CH) {
      const uint2 cm = nm, cv = nv;
      uint32_t acc[CH];
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < CH; ++j) acc[j] = nacc[j];
      if (c + CH < wcols) {
        tmem_ld_32x8(t_addr + (uint32_t)(c + CH), nacc);
        nm = ld_codes8(Mrow, c + CH, ncols, vec, 127u);
        nv = ld_codes8(Vrow, c + CH, ncols, vec, 0u);
      }
#pragma unroll
      for (int j = 0; j < CH; ++j) {
        const float r = __uint_as_float(acc[j]);
        const uint32_t im = ((j < 4 ? cm.x : cm.y) >> (8 * (j & 3))) & 0xffu, iv = ((j < 4 ? cv.x : cv.y) >> (8 * (j & 3))) & 0xffu;
        const float m = adam_m(__fmul_rn(t.code_s[im], am_m), r, ap);
        const float v = adam_v(__fmul_rn(t.code_u[iv], am_v), r, ap);
        mx_m = fmaxf(mx_m, fabsf(m));
        mx_vb = max(mx_vb, __float_as_uint(v));
      }
    }
  }
  for (int o = 1; o < p.q_rows; o <<= 1) {      // the q_rows lanes of the block (a power of two up to 32)
    mx_m = fmaxf(mx_m, __shfl_xor_sync(0xffffffffu, mx_m, o));
    mx_vb = max(mx_vb, __shfl_xor_sync(0xffffffffu, mx_vb, o));
  }
  const bool bad = mx_vb >= 0x7f800000u;
  const float mx_v = __uint_as_float(mx_vb);
  // an all-zero block: with 0 in place of the reciprocal every y' is 0 and takes the code of zero
  const float inv_m = mx_m != 0.f ? 1.0f / mx_m : 0.f, inv_v = mx_v != 0.f ? 1.0f / mx_v : 0.f;

  // ---- pass 2: N and the new codes, eight elements at a time with one (rare) branch to the exact search
  {
    uint2 nm = ld_codes8(Mrow, 0, ncols, vec, 127u), nv = ld_codes8(Vrow, 0, ncols, vec, 0u);
    uint32_t nacc[CH];
    tmem_ld_32x8(t_addr, nacc);
#pragma unroll 1
    for (int c = 0; c < wcols; c += CH) {
      const uint2 cm = nm, cv = nv;
      uint32_t acc[CH];
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < CH; ++j) acc[j] = nacc[j];
      if (c + CH < wcols) {
        tmem_ld_32x8(t_addr + (uint32_t)(c + CH), nacc);
        nm = ld_codes8(Mrow, c + CH, ncols, vec, 127u);
        nv = ld_codes8(Vrow, c + CH, ncols, vec, 0u);
      }
      float xm[CH], xv[CH];
      uint32_t nw[CH / 2];
#pragma unroll
      for (int j = 0; j < CH; j += 2) {
        float n[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int e = j + k;
          const float r = __uint_as_float(acc[e]);
          const uint32_t im = ((e < 4 ? cm.x : cm.y) >> (8 * (e & 3))) & 0xffu, iv = ((e < 4 ? cv.x : cv.y) >> (8 * (e & 3))) & 0xffu;
          xm[e] = adam_m(__fmul_rn(t.code_s[im], am_m), r, ap);
          xv[e] = adam_v(__fmul_rn(t.code_u[iv], am_v), r, ap);
          n[k] = adam_normalised(xm[e], xv[e], ap);
        }
        const __nv_bfloat162 h = __floats2bfloat162_rn(n[0], n[1]);
        nw[j >> 1] = *reinterpret_cast<const uint32_t*>(&h);
      }
      uint32_t pm[2] = {0u, 0u}, pv[2] = {0u, 0u}, need = 0u;     // need: bit e for M value e, bit 8 + e for V value e
#pragma unroll
      for (int e = 0; e < CH; ++e) {
        bool ex_m, ex_v;
        const uint32_t km = q8_encode_fast<true>(xm[e], inv_m, t.enc_s, ex_m) & 0xffu;
        const uint32_t kv = q8_encode_fast<false>(xv[e], inv_v, t.enc_u, ex_v) & 0xffu;
        pm[e >> 2] |= km << (8 * (e & 3));
        pv[e >> 2] |= kv << (8 * (e & 3));
        need |= ((ex_m ? 1u : 0u) << e) | ((ex_v ? 1u : 0u) << (8 + e));
      }
      if (need != 0u) {                         // about one value in 4000: the quotient by IEEE division, searched exactly
#pragma unroll
        for (int e = 0; e < CH; ++e) {
          if (need & (1u << e)) {
            const uint32_t k = (uint32_t)q8_encode(__fdiv_rn(xm[e], mx_m), t.mid_s) & 0xffu;
            pm[e >> 2] = (pm[e >> 2] & ~(0xffu << (8 * (e & 3)))) | (k << (8 * (e & 3)));
          }
          if (need & (0x100u << e)) {
            const uint32_t k = (uint32_t)q8_encode(__fdiv_rn(xv[e], mx_v), t.mid_u) & 0xffu;
            pv[e >> 2] = (pv[e >> 2] & ~(0xffu << (8 * (e & 3)))) | (k << (8 * (e & 3)));
          }
        }
      }
      if (vec) {
        *reinterpret_cast<uint2*>(Mrow + c) = make_uint2(pm[0], pm[1]);
        *reinterpret_cast<uint2*>(Vrow + c) = make_uint2(pv[0], pv[1]);
        *reinterpret_cast<uint4*>(Nrow + c) = make_uint4(nw[0], nw[1], nw[2], nw[3]);
      } else {
#pragma unroll
        for (int j = 0; j < CH; ++j)
          if (c + j < ncols) {
            Mrow[c + j] = (uint8_t)(pm[j >> 2] >> (8 * (j & 3)));
            Vrow[c + j] = (uint8_t)(pv[j >> 2] >> (8 * (j & 3)));
            reinterpret_cast<uint16_t*>(Nrow)[c + j] = (uint16_t)(nw[j >> 1] >> (16 * (j & 1)));
          }
      }
    }
  }
  if (ncols > 0 && (row % p.q_rows) == 0) {     // the first lane of each block stores its absmax
    p.Mam[tile] = mx_m;
    p.Vam[tile] = mx_v;
  }
  return bad;
}

// ---- the kernel -------------------------------------------------------------------------------

template <int EPI, typename TW, int CTAS>
__global__ void __launch_bounds__(epi_threads(EPI), 1)
gemm_tc_kernel(const __grid_constant__ TcGroup g) {
  using G = Geo<CTAS>;
  constexpr int kEpiWarps = epi_warps(EPI);
  constexpr int kStages = G::kStages;
  constexpr int kStageBytes = G::kStageBytes;
  extern __shared__ uint8_t smem_raw[];
  // stage ring, 1024-byte aligned for the 128-byte swizzle
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t ring = (raw_addr + 1023u) & ~1023u;
  uint8_t* ring_ptr = smem_raw + (ring - raw_addr);
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring_ptr + kStages * kStageBytes);
  // bars[0..S) full, [S..2S) empty, [2S..2S+2) accumulator full, [2S+2..2S+4) accumulator empty.
  // In a CTA pair the full and accumulator-empty barriers that count are the leader's (rank 0).
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto accf_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto acce_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + 2 * kStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * kStages + 5);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int total_units = g.unit_end[g.count - 1];
  const uint32_t rank = CTAS == 2 ? cluster_ctarank() : 0u;
  const int team = blockIdx.x / CTAS;               // CTA or CTA pair that walks the units together
  const int teams = gridDim.x / CTAS;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accf_bar(a), 1);
      mbar_init(acce_bar(a), kEpiWarps * CTAS);     // one arrival per epilogue warp of the group, from every CTA
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if (CTAS == 2) {
      tmem_alloc_pair(smem_u32((const void*)tmem_slot), kTmemCols);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(smem_u32((const void*)tmem_slot), kTmemCols);
      tmem_relinquish();
    }
  }
  // the 8-bit code tables follow the barriers (256 bytes after the ring)
  Q8Tables* q8t = reinterpret_cast<Q8Tables*>(ring_ptr + kStages * kStageBytes + 256);
  if constexpr (EPI == EPI_ADAM_Q8) q8_tables_fill(*q8t, g.q8, (int)threadIdx.x, epi_threads(EPI));
  tc_fence_before();
  __syncthreads();
  if (CTAS == 2) cluster_sync_all();                // the peer's barriers exist before anyone signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ================= TMA producer (every CTA loads its own share) =================
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      long long issued = 0;
      bool ok = true;
      for (int u = team; u < total_units && ok; u += teams) {
        int pi;
        const Unit w = decode_unit(g, u, pi);
        const bool A_MN = g.p[pi].a_mn != 0, B_MN = g.p[pi].b_mn != 0;
        const CUtensorMap* map_a = &g.map_a[pi];
        const CUtensorMap* map_b = &g.map_b[pi];
        const int m0 = w.m0 + (int)rank * kBM;               // this CTA's rows of A
        const int n0 = w.n0 + (int)rank * G::kBNcta;         // this CTA's columns of B
        for (int kb = w.kb_begin; kb < w.kb_end; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t a_dst = ring + stage * kStageBytes;
          const uint32_t b_dst = a_dst + kABytes;
          const uint32_t fbar = CTAS == 2 ? map_to_cta(full_bar(stage), 0) : full_bar(stage);
          if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), CTAS * kStageBytes);
          const int k0 = kb * kBK;
          auto load = [&](uint32_t dst, const CUtensorMap* map, int x, int y) {
            if (CTAS == 2) tma_load_2d_pair(dst, map, x, y, fbar);
            else tma_load_2d(dst, map, x, y, fbar);
          };
          if (A_MN) {
#pragma unroll
            for (int j = 0; j < kBM / 64; ++j) load(a_dst + j * (kBK * 128), map_a, m0 + 64 * j, k0);
          } else {
            load(a_dst, map_a, k0, m0);
          }
          if (B_MN) {
#pragma unroll
            for (int j = 0; j < G::kBNcta / 64; ++j) load(b_dst + j * (kBK * 128), map_b, n0 + 64 * j, k0);
          } else {
            load(b_dst, map_b, k0, n0);
          }
          ++issued;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && CTAS == 1) {
        // let the copies that are still in flight land before the CTA goes away
        int s = stage;
        uint32_t ph = phase;
        const long long pending = issued < kStages ? issued : kStages;
        for (long long i = 0; i < pending; ++i) {
          if (--s < 0) { s = kStages - 1; ph ^= 1u; }
          const long long t0 = clock64();
          while (!mbar_try_wait(full_bar(s), ph) && clock64() - t0 < kWaitLimitCycles) {}
        }
      }
    }
  } else if (warp == 1) {
    // ================= MMA issuer (the leader CTA of a pair issues for both) =================
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int u = team; u < total_units && ok; u += teams) {
        int pi;
        const Unit w = decode_unit(g, u, pi);
        const bool A_MN = g.p[pi].a_mn != 0, B_MN = g.p[pi].b_mn != 0;
        const uint32_t idesc = instr_desc(g.p[pi].a_mn, g.p[pi].b_mn, G::kTileM);
        if (!mbar_wait(acce_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kBN);
        for (int kb = w.kb_begin; kb < w.kb_end; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = ring + stage * kStageBytes;
          const uint32_t b_addr = a_addr + kABytes;
          const uint64_t a_desc = smem_desc(a_addr, A_MN);
          const uint64_t b_desc = smem_desc(b_addr, B_MN);
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            // K-major: 16 bf16 = 32 B along the swizzled row; MN-major: 16 k = two 8-k groups of 1024 B
            const uint64_t a_adv = (uint64_t)((A_MN ? k * 2048 : k * 32) >> 4);
            const uint64_t b_adv = (uint64_t)((B_MN ? k * 2048 : k * 32) >> 4);
            const uint32_t accum = (kb > w.kb_begin || k > 0) ? 1u : 0u;
            if (CTAS == 2) umma_bf16_pair(d_tmem, a_desc + a_adv, b_desc + b_adv, idesc, accum);
            else umma_bf16(d_tmem, a_desc + a_adv, b_desc + b_adv, idesc, accum);
          }
          // stage reusable (in both CTAs of a pair) once these MMAs have read it
          if (CTAS == 2) umma_commit_pair(empty_bar(stage));
          else umma_commit(empty_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) {                                     // accumulator complete
          if (CTAS == 2) umma_commit_pair(accf_bar(acc));
          else umma_commit(accf_bar(acc));
        }
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ================= epilogue =================
    const int quarter = warp & 3;                   // TMEM lanes 32*quarter .. +31 belong to this warp
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int u = team; u < total_units && ok; u += teams) {
      int pi;
      const Unit w = decode_unit(g, u, pi);
      const TcParams& p = g.p[pi];
      const int row = w.m0 + (int)rank * kBM + quarter * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * kBN);
      if constexpr (epi_is_adam(EPI)) {
        // warps 2..5 take the first 64 columns of the tile, warps 6..9 the next 64, and so on
        const int part = (warp - 2) >> 2;
        const int col0 = w.n0 + part * kAdamCols;
        bool bad;
        if constexpr (EPI == EPI_ADAM_F32)
          bad = epi_adam_f32(p, row, col0, t_row + (uint32_t)(part * kAdamCols), accf_bar(acc), acc_phase, abort_flag, ok);
        else
          bad = epi_adam_q8(p, row, col0, t_row + (uint32_t)(part * kAdamCols), accf_bar(acc), acc_phase, abort_flag, *q8t, ok);
        if (!ok) break;
        if (bad) atomicOr(p.status, GALORE_DEV_NONFINITE);
      } else if (EPI != EPI_PARTIAL && w.n0 + kBN <= p.N) {
        // Interior tile of the weight update.  The thread's stretch of its W row is fetched into
        // registers BEFORE waiting for the accumulator: the loads do not depend on the MMAs, so the
        // whole W tile streams in from HBM while the tensor cores are still working on it.
        constexpr int kVec = 16 / (int)sizeof(TW);            // elements per 16-byte vector
        constexpr int kPre = sizeof(TW) == 2 ? kBN : kBN / 2; // columns held in registers at once
        constexpr int kNV = kPre / kVec;                      // 32 vectors = 128 registers
        const bool row_ok = row < p.M;
        TW* wrow = (TW*)p.W + (int64_t)(row_ok ? row : 0) * p.ldw + w.n0;
        uint4 wv[kNV];
        const bool vec32 = p.vec32 != 0;
        auto fetch = [&](const TW* src) {
          if (vec32) {
#pragma unroll
            for (int j = 0; j < kNV; j += 2) ld_global_32B(reinterpret_cast<const uint4*>(src) + j, wv[j], wv[j + 1]);
          } else {
#pragma unroll
            for (int j = 0; j < kNV; ++j) wv[j] = reinterpret_cast<const uint4*>(src)[j];
          }
        };
        if (row_ok) fetch(wrow);
        if (!mbar_wait(accf_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int h = 0; h < kBN / kPre; ++h) {
          if (h > 0 && row_ok) fetch(wrow + h * kPre);
#pragma unroll
          for (int c = 0; c < kPre; c += 32) {
            uint32_t v[32];
            tmem_ld_32x32(t_row + (uint32_t)(h * kPre + c), v);
            tmem_ld_wait();
            if (row_ok) {
              uint4* dst = reinterpret_cast<uint4*>(wrow + h * kPre + c);
#pragma unroll
              for (int q = 0; q < 32 / kVec; ++q) apply_vec<TW, EPI == EPI_APPLY_DECAY>(wv[c / kVec + q], &v[q * kVec], p.scale, p.keep);
              if (vec32) {
#pragma unroll
                for (int q = 0; q < 32 / kVec; q += 2) st_global_32B(dst + q, wv[c / kVec + q], wv[c / kVec + q + 1]);
              } else {
#pragma unroll
                for (int q = 0; q < 32 / kVec; ++q) dst[q] = wv[c / kVec + q];
              }
            }
          }
        }
      } else {
        if (!mbar_wait(accf_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < kBN; c += 32) {
          if (w.n0 + c >= p.N) break;                 // columns past the matrix: nothing to write
          uint32_t v[32];
          tmem_ld_32x32(t_row + (uint32_t)c, v);
          tmem_ld_wait();
          if (EPI == EPI_PARTIAL) epi_partial(p, w, row, w.n0 + c, v);
          else epi_apply<TW, EPI == EPI_APPLY_DECAY>(p, row, w.n0 + c, v);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {                                // accumulator free for the MMA warp (the leader's)
        if (rank == 0) mbar_arrive(acce_bar(acc));
        else mbar_arrive_remote(map_to_cta(acce_bar(acc), 0));
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  if (CTAS == 2 && *abort_flag) {                     // gave up: let copies that are still in flight land
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {}
  }
  tc_fence_before();
  __syncthreads();
  if (CTAS == 2) cluster_sync_all();                  // neither CTA leaves while the peer may still signal it
  if (threadIdx.x == 0 && *abort_flag) atomicOr(g.p[0].status, GALORE_DEV_WAIT_EXPIRED);
  if (warp == 1) {
    tc_fence_after();
    if (CTAS == 2) tmem_dealloc_pair(tmem_base, kTmemCols);
    else tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---- host side --------------------------------------------------------------------------------------

PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;
std::mutex g_encode_mutex;

galore_status_t ensure_encode() {
  std::lock_guard<std::mutex> lock(g_encode_mutex);
  if (g_encode) return GALORE_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  GALORE_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
  if (!fn || qres != cudaDriverEntryPointSuccess) return GALORE_ERR_CUDA;
  g_encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
  return GALORE_OK;
}

// bf16 matrix, `rows` x `cols` (cols contiguous), leading dimension ld; box = box_rows x 64 columns, 128-byte swizzle
galore_status_t make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
  GALORE_TRY(ensure_encode());
  if (((uintptr_t)base & 15) || (ld * 2) % 16) return GALORE_ERR_ALIGNMENT;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    note_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return GALORE_ERR_CUDA;
  }
  return GALORE_OK;
}

int sm_count() {
  static int sms = 0;
  if (!sms) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  }
  return sms;
}

// Launches of these kernels given on different streams are chained with an event, in the order of
// the calls.  One CTA takes a whole SM's tensor memory and nearly all of its shared memory, so two
// of them never share an SM and little is lost; runs that kept several streams of them in flight
// did not finish on the test machines, and no cause was found in the code.
struct StreamChain {
  std::mutex mutex;
  cudaStream_t last[64] = {};
  cudaEvent_t done[64] = {};
  bool used[64] = {};
};
StreamChain g_chain;

galore_status_t chain_before(cudaStream_t st, int* dev_out) {
  int dev = 0;
  GALORE_CUDA_TRY(cudaGetDevice(&dev));
  *dev_out = dev;
  if (dev < 0 || dev >= 64) return GALORE_ERR_INVALID_ARG;
  if (g_chain.used[dev] && g_chain.last[dev] != st) GALORE_CUDA_TRY(cudaStreamWaitEvent(st, g_chain.done[dev], 0));
  return GALORE_OK;
}
galore_status_t chain_after(cudaStream_t st, int dev) {
  if (!g_chain.done[dev]) GALORE_CUDA_TRY(cudaEventCreateWithFlags(&g_chain.done[dev], cudaEventDisableTiming));
  GALORE_CUDA_TRY(cudaEventRecord(g_chain.done[dev], st));
  g_chain.last[dev] = st;
  g_chain.used[dev] = true;
  return GALORE_OK;
}

template <int EPI, typename TW, int CTAS>
galore_status_t launch_tc_variant(const TcGroup& g, cudaStream_t st) {
  auto kern = gemm_tc_kernel<EPI, TW, CTAS>;
  constexpr int smem = Geo<CTAS>::kSmemBytes + epi_smem(EPI);
  static_assert(smem <= 227 * 1024, "shared memory of one CTA");
  static bool configured = false;
  if (!configured) {
    GALORE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    configured = true;
  }
  const int units = g.unit_end[g.count - 1];
  if (units <= 0) return GALORE_OK;
  const int teams = std::min(units, sm_count() / CTAS);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(teams * CTAS));
  cfg.blockDim = dim3(epi_threads(EPI));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CTAS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  std::lock_guard<std::mutex> lock(g_chain.mutex);
  int dev = 0;
  GALORE_TRY(chain_before(st, &dev));
  GALORE_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, g));
  count_launch();
  return chain_after(st, dev);
}

// every problem of a group was tiled for the same variant (TcParams::tile_m)
template <int EPI, typename TW>
galore_status_t launch_tc(const TcGroup& g, cudaStream_t st) {
  if (g.count < 1 || g.count > kMaxGroup) return GALORE_ERR_INVALID_ARG;
  for (int i = 1; i < g.count; ++i)
    if (g.p[i].tile_m != g.p[0].tile_m) return GALORE_ERR_INVALID_ARG;
  if (g.p[0].tile_m == 2 * kBM) return launch_tc_variant<EPI, TW, 2>(g, st);
  return launch_tc_variant<EPI, TW, 1>(g, st);
}

// appends one problem to a group
void group_add(TcGroup& g, const CUtensorMap& ma, const CUtensorMap& mb, const TcParams& p) {
  const int i = g.count++;
  g.map_a[i] = ma;
  g.map_b[i] = mb;
  g.p[i] = p;
  g.unit_end[i] = (i > 0 ? g.unit_end[i - 1] : 0) + p.tiles_m * p.tiles_n * p.splits;
}

void fill_tiles(TcParams& p, int M, int N, int K, int splits, int ctas) {
  p.M = M; p.N = N; p.K = K;
  p.tile_m = kBM * ctas;
  p.tiles_m = (int)ceil_div(M, p.tile_m);
  p.tiles_n = (int)ceil_div(N, kBN);
  p.kblocks_total = (int)ceil_div(K, kBK);
  if (splits < 1) splits = 1;
  p.kblocks_per_split = (int)ceil_div(p.kblocks_total, splits);
  p.splits = (int)ceil_div(p.kblocks_total, p.kblocks_per_split);
}

// K slices that fill the last wave of CTAs best, keeping at least 4 k-blocks per slice
int choose_splits(int64_t M, int64_t N, int64_t K, int ctas) {
  const int64_t tiles = ceil_div(M, kBM * ctas) * ceil_div(N, kBN);
  const int kblocks = (int)ceil_div(K, kBK);
  const int sms = 148 / ctas;
  int best = 1;
  double best_score = -1.0;
  for (int s = 1; s <= 8; ++s) {
    const int per = (int)ceil_div(kblocks, s);
    if (s > 1 && per < 4) break;
    const int eff_s = (int)ceil_div(kblocks, per);
    if (eff_s != s) continue;
    const int64_t units = tiles * s;
    const double fill = (double)units / (double)(ceil_div(units, sms) * sms);
    // each extra slice costs one more partial buffer to write and read back
    const double score = fill - 0.02 * (s - 1);
    if (score > best_score + 1e-9) { best_score = score; best = s; }
  }
  return best;
}

}  // namespace

bool tensor_path_eligible(const galore_config_t& c) {
  return c.g_dtype == GALORE_BF16 && c.p_dtype == GALORE_BF16 && (c.rank % 8) == 0;
}

// CTA pairs (256-row tiles) whenever every GEMM of the layer has at least 256 rows
int tensor_ctas(const galore_config_t& c) { return c.rank >= 256 ? 2 : 1; }

int tensor_proj_splits(const galore_config_t& c, bool left) {
  const int ctas = tensor_ctas(c);
  if (left) return choose_splits(c.rank, c.n, c.m, ctas);
  return choose_splits(c.m, c.rank, c.n, ctas);
}

galore_status_t tensor_plan_init(TensorPlan* plan, const galore_config_t& c, bool left, void* P, void* Nbuf, float* Rpart,
                                 int splits, int64_t ld_part, int64_t ld_n) {
  plan->ready = false;
  plan->ctas = tensor_ctas(c);
  plan->splits = splits;
  plan->P = P;
  plan->Nbuf = Nbuf;
  plan->Rpart = Rpart;
  plan->ld_part = ld_part;
  plan->ld_n = ld_n;
  const int64_t r = c.rank;
  if (left) {
    // projection: A = P^T, MN-major from P (m x r);  back-projection: A = P, K-major
    GALORE_TRY(make_map(&plan->map_p_proj, P, c.m, r, r, 64));
    GALORE_TRY(make_map(&plan->map_p_back, P, c.m, r, r, kBM));
    // back-projection: B = N (r x n), MN-major
    GALORE_TRY(make_map(&plan->map_n_back, Nbuf, r, c.n, ld_n, 64));
  } else {
    // projection: B = Q (n x r), MN-major;  back-projection: B = Q^T, K-major from Q
    GALORE_TRY(make_map(&plan->map_p_proj, P, c.n, r, r, 64));
    GALORE_TRY(make_map(&plan->map_p_back, P, c.n, r, r, kBN / plan->ctas));   // each CTA of a pair stages half of B
    // back-projection: A = N (m x r), K-major
    GALORE_TRY(make_map(&plan->map_n_back, Nbuf, c.m, r, ld_n, kBM));
  }
  plan->ready = true;
  return GALORE_OK;
}

bool tensor_operands_aligned(const galore_config_t& c, const void* W, int64_t ldw, const void* G, int64_t ldg) {
  if (((uintptr_t)G & 15) || (ldg % 8)) return false;
  if ((uintptr_t)W & 15) return false;
  return c.w_dtype == GALORE_BF16 ? (ldw % 8) == 0 : (ldw % 4) == 0;
}

// ---- problems -----------------------------------------------------------------------------------

// R partials <- P^T G (left) / G Q (right)
static galore_status_t project_problem(const TensorPlan* plan, const galore_config_t& c, bool left, const void* G,
                                       int64_t ldg, float* part, int64_t ld_part, int splits, int32_t* status,
                                       TcParams* p, CUtensorMap* ma, CUtensorMap* mb) {
  if (!plan->ready) return GALORE_ERR_STATE;
  const int r = c.rank;
  *p = TcParams{};
  p->status = status;
  p->part = part;
  p->ld_part = ld_part;
  p->vec32 = (((uintptr_t)part & 31) == 0 && (ld_part % 8) == 0) ? 1 : 0;
  if (left) {
    // A = P^T, M/N-major from P; B = G, M/N-major.  G is the big operand: units sharing a G panel run together
    fill_tiles(*p, r, (int)c.n, (int)c.m, splits, plan->ctas);
    p->split_stride = (int64_t)r * ld_part;
    p->m_fast = 1;
    p->a_mn = 1;
    p->b_mn = 1;
    *ma = plan->map_p_proj;
    return make_map(mb, G, c.m, c.n, ldg, 64);
  }
  // A = G, K-major; B = Q, M/N-major
  fill_tiles(*p, (int)c.m, r, (int)c.n, splits, plan->ctas);
  p->split_stride = (int64_t)c.m * ld_part;
  p->m_fast = 0;
  p->a_mn = 0;
  p->b_mn = 1;
  *mb = plan->map_p_proj;
  return make_map(ma, G, c.m, c.n, ldg, kBM);
}

// the Adam part of a projection problem
static galore_status_t set_adam(TcParams* p, const TcAdamArgs& a) {
  if (a.state_fmt == GALORE_STATE_Q8_BLOCK &&
      (a.q_block < 256 || a.q_block > 2048 || (a.q_block & (a.q_block - 1)) != 0)) return GALORE_ERR_INVALID_ARG;
  p->Ms = a.M; p->Vs = a.V; p->Mc = a.Mc; p->Vc = a.Vc; p->Mam = a.Mam; p->Vam = a.Vam;
  p->ld_s = a.ld_s;
  p->q_rows = a.q_block / kStateTileCols;
  p->q_tiles_c = (int)ceil_div(p->N, kStateTileCols);
  p->Nout = (__nv_bfloat16*)a.Nout;
  p->ld_n = a.ld_n;
  p->ap = a.ap;
  // 32-byte accesses (16 for the code stores): per thread 64 bytes of codes, 64-byte runs of fp32 moments and
  // 32-byte runs of N, all starting at multiples of 16 columns
  const uintptr_t bases = (uintptr_t)a.Nout | (uintptr_t)a.M | (uintptr_t)a.V | (uintptr_t)a.Mc | (uintptr_t)a.Vc;
  const int64_t s_bytes = a.ld_s * (a.state_fmt == GALORE_STATE_F32 ? 4 : 1);
  p->adam_vec = ((bases & 31) == 0 && (s_bytes % 32) == 0 && (a.ld_n % 16) == 0) ? 1 : 0;
  return GALORE_OK;
}

static galore_status_t launch_project_adam(const TcGroup& g, int32_t state_fmt, cudaStream_t st) {
  if (state_fmt == GALORE_STATE_F32) return launch_tc<EPI_ADAM_F32, float>(g, st);
  return launch_tc<EPI_ADAM_Q8, float>(g, st);
}

// the weight update of a group: with the decay multiply only if some problem of the group decays
static galore_status_t launch_apply(const TcGroup& g, int32_t w_dtype, cudaStream_t st) {
  bool decay = false;
  for (int i = 0; i < g.count; ++i) decay = decay || g.p[i].keep != 1.0f;
  if (w_dtype == GALORE_BF16)
    return decay ? launch_tc<EPI_APPLY_DECAY, __nv_bfloat16>(g, st) : launch_tc<EPI_APPLY, __nv_bfloat16>(g, st);
  return decay ? launch_tc<EPI_APPLY_DECAY, float>(g, st) : launch_tc<EPI_APPLY, float>(g, st);
}

// W <- keep * W - scale * P N (left) / N Q^T (right); map_n addresses the normalised update
static galore_status_t back_problem(const TensorPlan* plan, const galore_config_t& c, bool left, const CUtensorMap& map_n,
                                    void* W, int64_t ldw, float scale, float keep, int32_t* status, TcParams* p,
                                    CUtensorMap* ma, CUtensorMap* mb) {
  if (!plan->ready) return GALORE_ERR_STATE;
  *p = TcParams{};
  p->status = status;
  p->W = W;
  p->ldw = ldw;
  p->vec32 = (((uintptr_t)W & 31) == 0 && (ldw * (int64_t)dtype_size(c.w_dtype)) % 32 == 0) ? 1 : 0;
  p->scale = scale;
  p->keep = keep;
  p->m_fast = 1;
  fill_tiles(*p, (int)c.m, (int)c.n, c.rank, 1, plan->ctas);
  if (left) {   // A = P K-major, B = N M/N-major
    p->a_mn = 0;
    p->b_mn = 1;
    *ma = plan->map_p_back;
    *mb = map_n;
  } else {      // A = N K-major, B = Q^T K-major from Q
    p->a_mn = 0;
    p->b_mn = 0;
    *ma = map_n;
    *mb = plan->map_p_back;
  }
  return GALORE_OK;
}

galore_status_t tensor_project(TensorPlan* plan, const galore_config_t& c, bool left, const void* G, int64_t ldg,
                               int32_t* status, cudaStream_t st) {
  TcParams p;
  CUtensorMap ma, mb;
  GALORE_TRY(project_problem(plan, c, left, G, ldg, plan->Rpart, plan->ld_part, plan->splits, status, &p, &ma, &mb));
  std::unique_ptr<TcGroup> g(new TcGroup);
  g->count = 0;
  group_add(*g, ma, mb, p);
  return launch_tc<EPI_PARTIAL, float>(*g, st);
}

galore_status_t tensor_project_adam(TensorPlan* plan, const galore_config_t& c, bool left, const void* G, int64_t ldg,
                                    const TcAdamArgs& adam, int32_t* status, cudaStream_t st) {
  TcParams p;
  CUtensorMap ma, mb;
  GALORE_TRY(project_problem(plan, c, left, G, ldg, nullptr, 0, 1, status, &p, &ma, &mb));
  GALORE_TRY(set_adam(&p, adam));
  std::unique_ptr<TcGroup> g(new TcGroup);
  g->count = 0;
  if (adam.state_fmt == GALORE_STATE_Q8_BLOCK) GALORE_TRY(q8_table_ptrs(&g->q8));
  group_add(*g, ma, mb, p);
  return launch_project_adam(*g, adam.state_fmt, st);
}

galore_status_t tensor_back_project(TensorPlan* plan, const galore_config_t& c, bool left, void* W, int64_t ldw,
                                    float scale, float keep, int32_t* status, cudaStream_t st) {
  TcParams p;
  CUtensorMap ma, mb;
  GALORE_TRY(back_problem(plan, c, left, plan->map_n_back, W, ldw, scale, keep, status, &p, &ma, &mb));
  std::unique_ptr<TcGroup> g(new TcGroup);
  g->count = 0;
  group_add(*g, ma, mb, p);
  return launch_apply(*g, c.w_dtype, st);
}

// ---- groups: many layers per launch ------------------------------------------------------------------

struct TensorGroup {
  TcGroup g;
};

TensorGroup* tensor_group_new() {
  TensorGroup* t = new (std::nothrow) TensorGroup;
  if (t) t->g.count = 0;
  return t;
}
void tensor_group_free(TensorGroup* t) { delete t; }
void tensor_group_reset(TensorGroup* t) { t->g.count = 0; }
int tensor_group_count(const TensorGroup* t) { return t->g.count; }
int tensor_group_capacity() { return kMaxGroup; }

galore_status_t tensor_group_add_project(TensorGroup* t, const TensorPlan* plan, const galore_config_t& c, bool left,
                                         const void* G, int64_t ldg, float* part, int64_t ld_part, int splits,
                                         int32_t* status) {
  if (t->g.count >= kMaxGroup) return GALORE_ERR_BUFFER_TOO_SMALL;
  TcParams p;
  CUtensorMap ma, mb;
  GALORE_TRY(project_problem(plan, c, left, G, ldg, part, ld_part, splits, status, &p, &ma, &mb));
  group_add(t->g, ma, mb, p);
  return GALORE_OK;
}

galore_status_t tensor_group_add_project_adam(TensorGroup* t, const TensorPlan* plan, const galore_config_t& c, bool left,
                                              const void* G, int64_t ldg, const TcAdamArgs& adam, int32_t* status) {
  if (t->g.count >= kMaxGroup) return GALORE_ERR_BUFFER_TOO_SMALL;
  TcParams p;
  CUtensorMap ma, mb;
  GALORE_TRY(project_problem(plan, c, left, G, ldg, nullptr, 0, 1, status, &p, &ma, &mb));
  GALORE_TRY(set_adam(&p, adam));
  group_add(t->g, ma, mb, p);
  return GALORE_OK;
}

galore_status_t tensor_group_launch_project_adam(TensorGroup* t, int32_t state_fmt, cudaStream_t st) {
  if (t->g.count == 0) return GALORE_OK;
  if (state_fmt == GALORE_STATE_Q8_BLOCK) GALORE_TRY(q8_table_ptrs(&t->g.q8));
  return launch_project_adam(t->g, state_fmt, st);
}

galore_status_t tensor_group_add_back(TensorGroup* t, const TensorPlan* plan, const galore_config_t& c, bool left,
                                      const void* Nbuf, int64_t ld_n, void* W, int64_t ldw, float scale, float keep,
                                      int32_t* status) {
  if (t->g.count >= kMaxGroup) return GALORE_ERR_BUFFER_TOO_SMALL;
  CUtensorMap map_n;
  if (left) GALORE_TRY(make_map(&map_n, Nbuf, c.rank, c.n, ld_n, 64));
  else GALORE_TRY(make_map(&map_n, Nbuf, c.m, c.rank, ld_n, kBM));
  TcParams p;
  CUtensorMap ma, mb;
  GALORE_TRY(back_problem(plan, c, left, map_n, W, ldw, scale, keep, status, &p, &ma, &mb));
  group_add(t->g, ma, mb, p);
  return GALORE_OK;
}

// A plain GEMM problem for the group: C (M x N, fp32, leading dimension ldc) = op(A) op(B), bf16
// operands.  a_mn = 1: A is stored K rows x M contiguous, 0: M rows x K contiguous; b_mn likewise
// (K x N contiguous resp. N x K contiguous).  All problems of a group must have M on the same side
// of 256 (they share the tile shape).
galore_status_t tensor_group_add_gemm(TensorGroup* t, const void* A, int64_t lda, int a_mn, const void* B, int64_t ldb,
                                      int b_mn, int M, int N, int K, float* C, int64_t ldc, int32_t* status) {
  if (t->g.count >= kMaxGroup) return GALORE_ERR_BUFFER_TOO_SMALL;
  const int ctas = M >= 2 * kBM ? 2 : 1;
  TcParams p = {};
  p.status = status;
  p.part = C;
  p.ld_part = ldc;
  p.split_stride = 0;
  p.vec32 = (((uintptr_t)C & 31) == 0 && (ldc % 8) == 0) ? 1 : 0;
  p.a_mn = a_mn ? 1 : 0;
  p.b_mn = b_mn ? 1 : 0;
  p.m_fast = 1;
  fill_tiles(p, M, N, K, 1, ctas);
  CUtensorMap ma, mb;
  if (a_mn) GALORE_TRY(make_map(&ma, A, K, M, lda, 64));
  else GALORE_TRY(make_map(&ma, A, M, K, lda, kBM));
  if (b_mn) GALORE_TRY(make_map(&mb, B, K, N, ldb, 64));
  else GALORE_TRY(make_map(&mb, B, N, K, ldb, kBN / ctas));
  group_add(t->g, ma, mb, p);
  return GALORE_OK;
}

galore_status_t tensor_group_launch_project(TensorGroup* t, cudaStream_t st) {
  if (t->g.count == 0) return GALORE_OK;
  return launch_tc<EPI_PARTIAL, float>(t->g, st);
}

galore_status_t tensor_group_launch_back(TensorGroup* t, int32_t w_dtype, cudaStream_t st) {
  if (t->g.count == 0) return GALORE_OK;
  return launch_apply(t->g, w_dtype, st);
}

}  // namespace galore
