// Grouped bf16 contraction on the 5th-generation tensor cores (sm_100a):
//   D_tile = sum over operand pairs p and k-blocks of A_p[128 x 64] * B_p[256 x 64]^T
// TMA (cp.async.bulk.tensor, 128-byte swizzle) stages operand tiles in shared memory, one elected
// thread issues tcgen05.mma (kind::f16, bf16 operands, fp32 accumulation) into tensor memory,
// four epilogue warps read the accumulator back with tcgen05.ld, turn it through shared memory so
// that global memory is accessed along rows, and apply a fused epilogue
// (factor EMA, bf16 hi/lo split, second-moment update, Adam scaling, weight write).
//
// A problem may sum several operand pairs into one tile (the bf16 hi/lo products of an fp32
// operand).  When the pairs are combinations of at most two distinct A and two distinct B operands
// (hi*hi + lo*hi + hi*lo), the kernel runs in its shared-operand form: a stage holds one k-block of
// every distinct operand (2 x 16 KiB + 2 x 32 KiB) and all combinations are issued from it, so each
// operand tile is fetched from L2 once per k-block instead of once per pair.
//
// One persistent CTA per SM walks a static tile list that spans every problem of a launch
// (all layers of one phase of the step), so small and large matrices share one launch.
// Two 256-column accumulators in tensor memory let the epilogue of a tile overlap the main
// loop of the next one.
//
// Operands may be K-major (K contiguous) or MN-major (M / N contiguous); the latter is how the
// row-major G, U, V enter products that contract over their row index (G^T G, U^T G, T V).
// Every tensor map is 3-D; the third coordinate selects a ring slot for operands that live in
// the stale-gradient ring and is 0 otherwise.
//
// Paired form (cta_group::2).  Two CTAs of a cluster, on neighbouring SMs, work on one 256 x 256
// tile: each stages its own 128 rows of A and only half of B (128 of the 256 result columns), the
// leader (cluster rank 0) issues tcgen05.mma.cta_group::2 of shape 256 x 256 x 16, which reads both
// halves of B from the two shared memories and leaves rows 0..127 of the accumulator in the leader's
// tensor memory and rows 128..255 in the peer's.  Per flop this takes two thirds of the L2 -> shared
// memory traffic and half of the shared-memory reads of B, which is what bounds the unpaired form.
// Barriers: both CTAs' TMA transactions complete on the leader's "full" barrier; the leader's
// commits arrive on the "empty" and "accumulator full" barriers of both CTAs (one commit per CTA, the
// peer's barrier addressed through mapa); the epilogue warps of both CTAs arrive on the leader's
// "accumulator empty" barrier.  Both CTAs meet at a cluster barrier after set-up and before they free
// their tensor memory, so neither exits while the other can still signal it.
//
// Folded form (factor products G G^T, G^T G).  The tensor core truncates its fp32 accumulator once
// per instruction (16-deep slice of the contraction), a one-sided error that grows with the length of
// the chain and with the size of the partial sums: 0.3 (K / 16) 2^-24 relative for contraction length
// K, 3e-6 at K = 2560.  The factors feed Power(), whose trailing basis vectors come out of a
// cancellation against eigenvalues 1e5 times larger, and an error of that size moves them by 1e-2.
// In this form the contraction is cut into chunks of a few k-blocks; the chunks are accumulated from
// zero, alternately in the two tensor-memory buffers, and eight epilogue warps (two per lane quadrant,
// 128 result columns each) add every finished chunk, round to nearest on the CUDA cores, to a running
// sum they keep in registers, while the tensor core is already working on the next chunk.  Chains
// are 8 to 16 instructions on partial sums a tenth the size: the error drops by the number of chunks.
// The final epilogue (factor EMA and its mirror image) runs from the registers while the first two
// chunks of the next tile accumulate.
//
// Every wait on an mbarrier is bounded: when a wait gives up the CTA raises an abort flag,
// records BR_ERR_TIMEOUT in the status word, leaves its loops, frees its tensor memory and
// returns; later launches return at once while the status word is negative.
#include <cuda.h>

#include <cstdlib>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

#include "br_internal.h"

namespace br {

namespace {

constexpr int BM = 128, BN = 256, BK = 64;       // tile (elements); BK*2 bytes = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;             // 16 KiB
constexpr int B_BYTES = BN * BK * 2;             // 32 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int SH_STAGES = 2;                     // shared-operand form: two stages of 2 A tiles + 2 B tiles
constexpr int SH_STAGE_BYTES = 2 * A_BYTES + 2 * B_BYTES;
static_assert(SH_STAGES * SH_STAGE_BYTES == STAGES * STAGE_BYTES, "both forms use the same operand area");
constexpr int EPI_LD = 33;                       // padded row of an epilogue tile (floats): rows and columns both conflict-free
constexpr int EPI_BYTES = 4 * 32 * EPI_LD * 4;   // one 32 x 32 fp32 tile per epilogue warp
constexpr int OPERAND_BYTES = STAGES * STAGE_BYTES;                   // 192 KiB of operand stages in every form
constexpr int SMEM_BYTES = OPERAND_BYTES + EPI_BYTES + 1024;          // + slack to align the tiles to 1 KiB
constexpr int MAX_STAGES = 6;
// Per-form geometry.  PAIR: the CTA pair owns a 256-row tile, each CTA stages 128 columns of B.
template <bool SHARED, bool PAIR>
struct Form {
  static constexpr int TM = PAIR ? 2 * BM : BM;                 // rows of a tile
  static constexpr int BNC = PAIR ? BN / 2 : BN;                // result columns whose B rows this CTA stages
  static constexpr int BB = BNC * BK * 2;                       // bytes of one staged B tile
  static constexpr int STAGE = SHARED ? 2 * A_BYTES + 2 * BB : A_BYTES + BB;
  static constexpr int NST = OPERAND_BYTES / STAGE;             // 4 / 2 unpaired, 6 / 3 paired
  static_assert(NST <= MAX_STAGES && NST * STAGE == OPERAND_BYTES, "stages fill the operand area");
};
constexpr int TMEM_COLS = 512;
constexpr int NUM_THREADS = 192;                 // warp 0: TMA, warp 1: MMA, warps 2..5: epilogue
constexpr int FOLD_THREADS = 320;                // folded form: warps 2..9 fold and write (two per lane quadrant)
constexpr int SMEM_BYTES_FOLD = OPERAND_BYTES + 2 * EPI_BYTES + 1024;
constexpr int MAX_PAIRS = 3;
// Tile rasterisation: a group of row-blocks (or, transposed, of column-blocks) is swept across the
// other dimension, so that the group's operand panel stays in L2 while the other operand streams
// through once per group.  The host picks orientation and group size per problem (see plan creation).
constexpr double kL2PanelBytes = 40e6;           // what one resident operand panel may take of the 126 MB L2

struct alignas(128) DevProblem {
  CUtensorMap mapA[MAX_PAIRS];
  CUtensorMap mapB[MAX_PAIRS];
  int32_t Md, Nd, K, n_pairs;
  int32_t a_mn, b_mn, epilogue, tiles_m;
  int32_t tiles_n, tile_begin, tile_count, tau_max;
  int32_t ring_slots, a_ring_mask, b_ring_mask, dyn_scalars;
  float alpha, beta, eps, beta1;
  float* D;
  long long ldd;
  __nv_bfloat16* Dh;
  __nv_bfloat16* Dl;
  long long ldh;
  float* D2;
  // shared-operand form: mapA[0..nA) / mapB[0..nB) are the distinct operands, `combos` lists the
  // products to issue per k-block: bits 8.. = count, bits 2c, 2c+1 = (A index, B index) of product c
  int32_t symmetric, nA, nB, combos;
  int32_t group, raster_n;        // blocks per group; 0: groups of row-blocks, 1: groups of column-blocks
  int32_t tri;                    // symmetric product with square tiles: the tile list holds the upper triangle only
  const float* clip;              // clipping factors by call (see TcProblem::clip_mode), or null
  int32_t clip_slots, clip_mode;
  int32_t fold_kb;                // folded form: k-blocks per chunk
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
// the same with cluster scope: the barrier also receives arrivals from the other CTA of a pair
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t ld_cluster_u32(uint32_t cluster_addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(cluster_addr) : "memory");
  return v;
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

constexpr uint64_t kWaitLimitNs = 2000000000ull;   // 2 s: far above any legitimate wait

// Bounded wait.  Returns false when the wait gave up or another role raised the abort flag.
template <bool CLUSTER = false>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int* status, uint64_t limit_ns = kWaitLimitNs) {
  auto try_wait = [&] { return CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity); };
  if (try_wait()) return true;
  const uint64_t t0 = global_timer_ns();
  uint32_t spins = 0;
  while (true) {
    if (try_wait()) return true;
    if ((++spins & 0xFF) == 0) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > limit_ns) {
        *abort_flag = 1;
        atomicMin(status, (int)BR_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}

// paired form: the transaction completes on `bar`, a shared::cluster address that may lie in the leader CTA
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                                 int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// paired form: `bar` is a shared::cluster address (this CTA's barrier or the peer's)
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Arrive on an mbarrier once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
         "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
         "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
         "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle.  lbo / sbo in bytes.
//   K-major : rows of 128 bytes (64 elements of K); 8-row groups 1024 bytes apart (sbo); lbo unused.
//   MN-major: rows of 128 bytes (64 elements of M/N), one row per k; 8-k groups sbo apart,
//             64-element M/N blocks lbo apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;     // descriptor version of this architecture
  d |= 2ull << 61;     // 128-byte swizzle
  return d;
}

// Instruction descriptor of kind::f16: fp32 accumulator, bf16 A and B, M = 128, N = 256.
__device__ __forceinline__ uint32_t make_idesc(int a_mn, int b_mn, int rows = BM) {
  uint32_t d = 0;
  d |= 1u << 4;                       // accumulator format: fp32
  d |= 1u << 7;                       // A format: bf16
  d |= 1u << 10;                      // B format: bf16
  d |= (uint32_t)(a_mn ? 1 : 0) << 15;
  d |= (uint32_t)(b_mn ? 1 : 0) << 16;
  d |= (uint32_t)(BN >> 3) << 17;
  d |= (uint32_t)(rows >> 4) << 24;
  return d;
}

__device__ __forceinline__ uint32_t pack2_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

struct TileInfo {
  const DevProblem* p;
  int m0, n0, z;
  bool active;
};

// tile index -> problem (binary search over tile_begin) and block coordinates
template <int TM>
__device__ __forceinline__ TileInfo locate_tile(const DevProblem* probs, int n_probs, int tile,
                                                long long calls, int tau) {
  int lo = 0, hi = n_probs - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (probs[mid].tile_begin <= tile) lo = mid; else hi = mid - 1;
  }
  const DevProblem* p = probs + lo;
  TileInfo ti;
  ti.p = p;
  const int local = tile - p->tile_begin;
  if (p->tri) {
    // upper triangle, column by column: column c holds the row-blocks 0..c at positions c (c + 1) / 2 + r
    int c = (int)((sqrtf(8.0f * (float)local + 1.0f) - 1.0f) * 0.5f);
    while ((c + 1) * (c + 2) / 2 <= local) ++c;
    while (c * (c + 1) / 2 > local) --c;
    ti.m0 = (local - c * (c + 1) / 2) * TM;
    ti.n0 = c * BN;
    const int tl = tau < 0 ? p->tau_max : tau;
    ti.active = (calls - tl >= 1);
    ti.z = 0;
    if (p->ring_slots > 0 && ti.active) ti.z = (int)((calls - 1 - tl) % p->ring_slots);
    return ti;
  }
  const int g = p->group;
  const int across = p->raster_n ? p->tiles_m : p->tiles_n;      // blocks of the swept dimension
  const int along = p->raster_n ? p->tiles_n : p->tiles_m;       // blocks of the grouped dimension
  const int per_group = g * across;
  const int group = local / per_group;
  const int first = group * g;
  const int gsz = min(along - first, g);
  const int in_group = local - group * per_group;
  const int blk_g = first + in_group % gsz, blk_s = in_group / gsz;
  ti.m0 = (p->raster_n ? blk_s : blk_g) * TM;
  ti.n0 = (p->raster_n ? blk_g : blk_s) * BN;
  // delayed-gradient bookkeeping: the layer is active once call - tau >= 1; the gradient to
  // apply sits in ring slot (calls - 1 - tau) mod slots
  const int tl = tau < 0 ? p->tau_max : tau;
  ti.active = (calls - tl >= 1);
  // a symmetric product is computed on the tiles that touch the upper triangle only
  if (p->symmetric && ti.m0 >= ti.n0 + BN) ti.active = false;
  ti.z = 0;
  if (p->ring_slots > 0 && ti.active) ti.z = (int)((calls - 1 - tl) % p->ring_slots);
  return ti;
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
template <bool SHARED, bool PAIR, bool FOLD = false>
__global__ void __launch_bounds__(FOLD ? FOLD_THREADS : NUM_THREADS, 1)
k_tc_gemm(const DevProblem* __restrict__ probs, int n_probs, int first_tile, int total_tiles, long long calls,
          int tau, float dyn_alpha, float dyn_beta, int* status) {
  using F = Form<SHARED, PAIR>;
  constexpr int NST = F::NST;
  constexpr int TM = F::TM;
  extern __shared__ uint8_t smem_raw[];
  __shared__ alignas(8) uint64_t bars[2 * MAX_STAGES + 4];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_word;
  __shared__ uint32_t dead_word;
  volatile int* abort_flag = &abort_word;

  // an earlier launch failed: nothing to do (a pair takes the decision from its leader, below)
  if (!PAIR && *reinterpret_cast<volatile int*>(status) < 0) return;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;        // 0: leader of the pair
  const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;      // index of this CTA (pair) in the tile walk
  const int n_units = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  // operand slot i of stage s
  auto sA = [&](int s, int i) {
    return SHARED ? tiles_base + (uint32_t)s * F::STAGE + (uint32_t)i * A_BYTES
                  : tiles_base + (uint32_t)s * A_BYTES;
  };
  auto sB = [&](int s, int i) {
    return SHARED ? tiles_base + (uint32_t)s * F::STAGE + 2u * A_BYTES + (uint32_t)i * F::BB
                  : tiles_base + (uint32_t)NST * A_BYTES + (uint32_t)s * F::BB;
  };
  float* epi_tiles = reinterpret_cast<float*>(smem_raw + ((tiles_base - smem_u32(smem_raw)) + (uint32_t)OPERAND_BYTES));
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (MAX_STAGES + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * MAX_STAGES + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * MAX_STAGES + 2 + a); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < NST; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    // accumulator hand-back: four epilogue warps, of both CTAs in the paired form
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), (FOLD ? 2 : 1) * (PAIR ? 8 : 4)); }
    abort_word = 0;
    dead_word = (*reinterpret_cast<volatile int*>(status) < 0) ? 1u : 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (PAIR) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  bool dead = false;
  if (PAIR) {
    // both CTAs have initialised their barriers before either signals the other; the pair skips its
    // work together when the leader saw a failed status word
    cluster_barrier();
    dead = ld_cluster_u32(map_to_cta(smem_u32(&dead_word), 0)) != 0u;
  }
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  if (dead) first_tile = total_tiles;          // every role finds an empty tile list

  if (warp == 0) {
    // ======================= TMA producer =======================
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      // paired form: the CTA's own rows of A and its half of the rows of B; every transaction of
      // the pair completes on the leader's barrier, on which only the leader posts the byte count
      const int row_off = (int)rank * BM, col_off = (int)rank * F::BNC;
      auto load = [&](uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
        if (PAIR) tma_load_3d_pair(dst, map, bar, x, y, z); else tma_load_3d(dst, map, bar, x, y, z);
      };
      for (int tile = first_tile + unit; tile < total_tiles && !*abort_flag; tile += n_units) {
        const TileInfo ti = locate_tile<TM>(probs, n_probs, tile, calls, tau);
        if (!ti.active) continue;
        const DevProblem* p = ti.p;
        const int nkb = (p->K + BK - 1) / BK;
        bool ok = true;
        auto load_a = [&](uint32_t dst, const CUtensorMap* ma, int k0, int za, uint32_t bar) {
          if (p->a_mn) {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j) load(dst + j * (BK * 128), ma, bar, ti.m0 + row_off + 64 * j, k0, za);
          } else {
            load(dst, ma, bar, k0, ti.m0 + row_off, za);
          }
        };
        auto load_b = [&](uint32_t dst, const CUtensorMap* mb, int k0, int zb, uint32_t bar) {
          if (p->b_mn) {
#pragma unroll
            for (int j = 0; j < F::BNC / 64; ++j) load(dst + j * (BK * 128), mb, bar, ti.n0 + col_off + 64 * j, k0, zb);
          } else {
            load(dst, mb, bar, k0, ti.n0 + col_off, zb);
          }
        };
        const uint32_t copies = PAIR ? 2u : 1u;
        if (SHARED) {
          for (int kb = 0; kb < nkb; ++kb) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, status)) { ok = false; break; }
            const uint32_t fb = PAIR ? map_to_cta(full_bar(stage), 0) : full_bar(stage);
            if (rank == 0) mbar_expect_tx(full_bar(stage), copies * (uint32_t)(p->nA * A_BYTES + p->nB * F::BB));
            for (int i = 0; i < p->nA; ++i)
              load_a(sA(stage, i), &p->mapA[i], kb * BK, ((p->a_ring_mask >> i) & 1) ? ti.z : 0, fb);
            for (int i = 0; i < p->nB; ++i)
              load_b(sB(stage, i), &p->mapB[i], kb * BK, ((p->b_ring_mask >> i) & 1) ? ti.z : 0, fb);
            if (++stage == NST) { stage = 0; phase ^= 1u; }
          }
        } else {
          for (int pr = 0; pr < p->n_pairs && ok; ++pr) {
            const int za = ((p->a_ring_mask >> pr) & 1) ? ti.z : 0;
            const int zb = ((p->b_ring_mask >> pr) & 1) ? ti.z : 0;
            for (int kb = 0; kb < nkb; ++kb) {
              if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, status)) { ok = false; break; }
              const uint32_t fb = PAIR ? map_to_cta(full_bar(stage), 0) : full_bar(stage);
              if (rank == 0) mbar_expect_tx(full_bar(stage), copies * (uint32_t)F::STAGE);
              load_a(sA(stage, 0), &p->mapA[pr], kb * BK, za, fb);
              load_b(sB(stage, 0), &p->mapB[pr], kb * BK, zb, fb);
              if (++stage == NST) { stage = 0; phase ^= 1u; }
            }
          }
        }
        if (!ok) break;
      }
    }
  } else if (warp == 1) {
    // ======================= MMA issuer =======================
    // (paired form: the leader issues for both CTAs; the peer's warp only owns the tensor-memory allocation)
    if (lane == 0 && rank == 0) {
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      uint32_t fold_seq = 0;                      // folded form: chunks handed over so far (buffer = seq & 1)
      // a commit arrives on this CTA's barrier and, in the paired form, on the peer's as well
      auto commit = [&](uint32_t bar) {
        if (PAIR) { umma_commit_pair(bar); umma_commit_pair(map_to_cta(bar, 1)); } else { umma_commit(bar); }
      };
      for (int tile = first_tile + unit; tile < total_tiles && !*abort_flag; tile += n_units) {
        const TileInfo ti = locate_tile<TM>(probs, n_probs, tile, calls, tau);
        if (!ti.active) continue;
        const DevProblem* p = ti.p;
        const int nkb = (p->K + BK - 1) / BK;
        const uint32_t idesc = make_idesc(p->a_mn, p->b_mn, TM);
        // K-major: advance 32 bytes per 16-element k step inside the swizzle row;
        // MN-major: 16 k rows = two 8-row groups of 1024 bytes.
        const uint32_t a_lbo = p->a_mn ? BK * 128 : 0, a_adv = p->a_mn ? 2048 : 32;
        const uint32_t b_lbo = p->b_mn ? BK * 128 : 0, b_adv = p->b_mn ? 2048 : 32;
        if (FOLD) {
          // chunks of fold_kb k-blocks, each accumulated from zero, alternately in the two buffers, and
          // handed to the epilogue warps, which add it to the running sum in their registers
          bool ok = true;
          for (int kb0 = 0; kb0 < nkb && ok; kb0 += p->fold_kb) {
            const int buf = (int)(fold_seq & 1u);
            if (!mbar_wait<PAIR>(tempty_bar(buf), ((fold_seq >> 1) & 1u) ^ 1u, abort_flag, status)) { ok = false; break; }
            tc_fence_after();
            const uint32_t d_chunk = tmem_base + (uint32_t)buf * BN;
            uint32_t accumulate = 0;
            const int kb1 = min(nkb, kb0 + p->fold_kb);
            for (int kb = kb0; kb < kb1; ++kb) {
              if (!mbar_wait(full_bar(stage), phase, abort_flag, status)) { ok = false; break; }
              tc_fence_after();
              const uint64_t adesc = make_smem_desc(sA(stage, 0), a_lbo, 1024);
              const uint64_t bdesc = make_smem_desc(sB(stage, 0), b_lbo, 1024);
#pragma unroll
              for (int k = 0; k < BK / UMMA_K; ++k) {
                if (PAIR)
                  umma_bf16_pair(d_chunk, adesc + (uint64_t)((k * a_adv) >> 4), bdesc + (uint64_t)((k * b_adv) >> 4),
                                 idesc, accumulate);
                else
                  umma_bf16(d_chunk, adesc + (uint64_t)((k * a_adv) >> 4), bdesc + (uint64_t)((k * b_adv) >> 4),
                            idesc, accumulate);
                accumulate = 1;
              }
              commit(empty_bar(stage));
              if (++stage == NST) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
            commit(tfull_bar(buf));
            ++fold_seq;
          }
          if (!ok) break;
          continue;
        }
        if (!mbar_wait<PAIR>(tempty_bar(acc), acc_phase ^ 1u, abort_flag, status)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
        uint32_t accumulate = 0;
        bool ok = true;
        const int n_steps = SHARED ? nkb : p->n_pairs * nkb;
        const int n_combo = SHARED ? (p->combos >> 8) : 1;
        for (int it = 0; it < n_steps; ++it) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          for (int c = 0; c < n_combo; ++c) {
            const int ai = SHARED ? ((p->combos >> (2 * c)) & 1) : 0;
            const int bi = SHARED ? ((p->combos >> (2 * c + 1)) & 1) : 0;
            const uint64_t adesc = make_smem_desc(sA(stage, ai), a_lbo, 1024);
            const uint64_t bdesc = make_smem_desc(sB(stage, bi), b_lbo, 1024);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
              if (PAIR)
                umma_bf16_pair(d_tmem, adesc + (uint64_t)((k * a_adv) >> 4), bdesc + (uint64_t)((k * b_adv) >> 4),
                               idesc, accumulate);
              else
                umma_bf16(d_tmem, adesc + (uint64_t)((k * a_adv) >> 4), bdesc + (uint64_t)((k * b_adv) >> 4),
                          idesc, accumulate);
              accumulate = 1;
            }
          }
          commit(empty_bar(stage));               // frees the stage once these MMAs have read it
          if (++stage == NST) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        commit(tfull_bar(acc));                   // accumulator complete
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    // ======================= epilogue warps =======================
    // A warp may read only its own quadrant of tensor memory, where lane = accumulator row: a
    // 32 x 32 block arrives with one row per lane.  It is turned through a padded shared-memory
    // tile so that global memory is accessed along rows: 8 lanes cover 128 contiguous bytes of one
    // row, a warp instruction four whole rows.  The values a read-modify-write epilogue needs are
    // prefetched into L2 while the main loop of the tile is still running and then loaded eight
    // rows deep before the first one is used.  A symmetric product (the factor EMAs) writes its
    // strictly-upper blocks a second time, transposed, instead of computing the lower triangle.
    const int quad = warp & 3;                    // tensor-memory lane quadrant this warp may read
    float* tile = epi_tiles + quad * (32 * EPI_LD);
    const int sub_r = lane >> 3, sub_c = (lane & 7) * 4;
    int acc = 0; uint32_t acc_phase = 0;
    uint32_t fold_seq = 0;
    for (int tile_i = first_tile + unit; tile_i < total_tiles && !*abort_flag; tile_i += n_units) {
      const TileInfo ti = locate_tile<TM>(probs, n_probs, tile_i, calls, tau);
      if (!ti.active) continue;
      const DevProblem* p = ti.p;
      float alpha = p->dyn_scalars ? dyn_alpha : p->alpha;
      const float beta = p->dyn_scalars ? dyn_beta : p->beta;
      const float eps = p->eps;
      const int epi = p->epilogue;
      // clipping factor of the call whose gradient this accumulator was built from
      float gclip = 1.0f;
      if (p->clip) {
        const int tl = tau < 0 ? p->tau_max : tau;
        gclip = p->clip[(int)((calls - 1 - tl) % p->clip_slots)];
        if (p->clip_mode == 2) alpha *= gclip * gclip;
      }
      const int row_base = ti.m0 + (int)rank * BM + quad * 32;
      const bool quad_ok = row_base < p->Md;      // uniform across the warp
      const bool reads_d = (epi == EPI_AXPBY_F32 && beta != 0.0f) || epi == EPI_ROTATED_ADAM ||
                           epi == EPI_SECOND_MOMENT || epi == EPI_SCALE_BF16;
      if (reads_d && row_base + lane < p->Md) {
        const float* d = p->D + (long long)(row_base + lane) * p->ldd + ti.n0;
#pragma unroll
        for (int q = 0; q < BN / 32; ++q)
          if (ti.n0 + 32 * q < p->Nd) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(d + 32 * q));
            if (epi == EPI_ROTATED_ADAM)
              asm volatile("prefetch.global.L2 [%0];" ::"l"(p->D2 + (long long)(row_base + lane) * p->ldd + ti.n0 + 32 * q));
          }
      }
      if (FOLD) {
        // ---- folded form: this warp owns 32 rows (its lane quadrant) x 128 columns (its half) ----
        const int half = (warp - 2) >> 2;
        float* ftile = epi_tiles + (warp - 2) * (32 * EPI_LD);
        const int nkb = (p->K + BK - 1) / BK;
        const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(half * 128);
        // which of the four 32-column blocks are written at all (uniform across the warp)
        uint32_t need = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const int col0 = ti.n0 + half * 128 + 32 * b;
          if (col0 < p->Nd && quad_ok && !(p->symmetric && row_base >= col0 + 32)) need |= 1u << b;
        }
        // The running sum of this thread: its row, its warp's 128 columns.  The first chunk is loaded
        // straight into these registers; every later one is added with packed fp32 adds, one 32-column
        // block at a time (the other warp of the quadrant covers the load latency).
        uint32_t sum[4][32];
        bool ok = true;
        for (int kb0 = 0; kb0 < nkb; kb0 += p->fold_kb) {
          const int buf = (int)(fold_seq & 1u);
          if (!mbar_wait(tfull_bar(buf), (fold_seq >> 1) & 1u, abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t src = lane_base + (uint32_t)(buf * BN);
          if (kb0 == 0) {
#pragma unroll
            for (int b = 0; b < 4; ++b)
              if ((need >> b) & 1u) tmem_ld32_issue(src + 32 * b, sum[b]);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int b = 0; b < 4; ++b) {
              if (!((need >> b) & 1u)) continue;
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                uint32_t t[16];
                tmem_ld16_issue(src + 32 * b + 16 * h, t);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                  const float2 r = __fadd2_rn(make_float2(__uint_as_float(sum[b][16 * h + j]), __uint_as_float(sum[b][16 * h + j + 1])),
                                              make_float2(__uint_as_float(t[j]), __uint_as_float(t[j + 1])));
                  sum[b][16 * h + j] = __float_as_uint(r.x); sum[b][16 * h + j + 1] = __float_as_uint(r.y);
                }
              }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            if (PAIR) mbar_arrive_cluster(map_to_cta(tempty_bar(buf), 0)); else mbar_arrive(tempty_bar(buf));
          }
          ++fold_seq;
        }
        if (!ok) break;
        // ---- factor EMA D <- alpha sum + beta D on the blocks that touch the upper triangle, and their mirror image ----
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          if (!((need >> b) & 1u)) continue;
          const int col0 = ti.n0 + half * 128 + 32 * b;
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 32; ++j) ftile[lane * EPI_LD + j] = __uint_as_float(sum[b][j]);
          __syncwarp();
          const int col = col0 + sub_c;
          int n_it = 0;
          if (col < p->Nd) { n_it = (p->Md - row_base - sub_r + 3) >> 2; n_it = n_it > 8 ? 8 : n_it; }
          float* d = p->D + (long long)(row_base + sub_r) * p->ldd + col;
          const long long step = 4 * p->ldd;
          const bool mirror = p->symmetric && col0 >= row_base + 32;
          // four row groups at a time (registers): read the old values, combine, write, and put the
          // result back into the tile for the mirror image
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float4 o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
              if (beta != 0.0f && 4 * h + i < n_it) o[i] = *reinterpret_cast<const float4*>(d + (4 * h + i) * step);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int it = 4 * h + i;
              float* t4 = ftile + (it * 4 + sub_r) * EPI_LD + sub_c;
              float4 r = make_float4(alpha * t4[0], alpha * t4[1], alpha * t4[2], alpha * t4[3]);
              if (beta != 0.0f && it < n_it) {
                r.x = fmaf(beta, o[i].x, r.x); r.y = fmaf(beta, o[i].y, r.y);
                r.z = fmaf(beta, o[i].z, r.z); r.w = fmaf(beta, o[i].w, r.w);
              }
              if (it < n_it) *reinterpret_cast<float4*>(d + it * step) = r;
              if (mirror) { t4[0] = r.x; t4[1] = r.y; t4[2] = r.z; t4[3] = r.w; }     // (each thread rewrites only what it read)
            }
          }
          if (mirror) {
            __syncwarp();
            const int mrow0 = col0 + sub_r, mcol = row_base + sub_c;
            if (mcol < p->Nd) {
#pragma unroll
              for (int it = 0; it < 8; ++it) {
                const int mrow = mrow0 + it * 4;
                if (mrow >= p->Md) break;
                const float* t1 = ftile + sub_c * EPI_LD + (it * 4 + sub_r);
                *reinterpret_cast<float4*>(p->D + (long long)mrow * p->ldd + mcol) =
                    make_float4(t1[0], t1[EPI_LD], t1[2 * EPI_LD], t1[3 * EPI_LD]);
              }
            }
          }
        }
        continue;
      }
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, status)) break;
      tc_fence_after();
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        const int col0 = ti.n0 + c0;
        if (col0 >= p->Nd) break;                 // uniform across the warp
        float v[32];
        tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN + c0), v);
        // nothing to write: rows beyond the matrix, or a block strictly below the diagonal of a
        // symmetric product (its mirror image is written by the block above the diagonal)
        if (!quad_ok || (p->symmetric && row_base >= col0 + 32)) continue;
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 32; ++j) tile[lane * EPI_LD + j] = v[j];
        __syncwarp();
        const int col = col0 + sub_c;
        // columns come in multiples of 8: a group of four is all in or all out
        int n_it = 0;
        if (col < p->Nd) { n_it = (p->Md - row_base - sub_r + 3) >> 2; n_it = n_it > 8 ? 8 : n_it; }
        float4 a[8];
#pragma unroll
        for (int it = 0; it < 8; ++it) {
          const float* t4 = tile + (it * 4 + sub_r) * EPI_LD + sub_c;
          a[it] = make_float4(t4[0], t4[1], t4[2], t4[3]);
        }
        if (epi == EPI_AXPBY_F32) {
          float* d = p->D + (long long)(row_base + sub_r) * p->ldd + col;
          const long long step = 4 * p->ldd;
          float4 old[8];
          if (beta != 0.0f) {
#pragma unroll
            for (int it = 0; it < 8; ++it)
              if (it < n_it) old[it] = *reinterpret_cast<const float4*>(d + it * step);
          }
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            float4 o = make_float4(alpha * a[it].x, alpha * a[it].y, alpha * a[it].z, alpha * a[it].w);
            if (beta != 0.0f && it < n_it) {
              o.x = fmaf(beta, old[it].x, o.x); o.y = fmaf(beta, old[it].y, o.y);
              o.z = fmaf(beta, old[it].z, o.z); o.w = fmaf(beta, old[it].w, o.w);
            }
            if (it < n_it) *reinterpret_cast<float4*>(d + it * step) = o;
            a[it] = o;
          }
          if (p->symmetric && col0 >= row_base + 32) {
            // mirror image: element (r, c) of this block also is element (c, r) of the result
            __syncwarp();
#pragma unroll
            for (int it = 0; it < 8; ++it) {
              float* t4 = tile + (it * 4 + sub_r) * EPI_LD + sub_c;
              t4[0] = a[it].x; t4[1] = a[it].y; t4[2] = a[it].z; t4[3] = a[it].w;
            }
            __syncwarp();
            const int mrow0 = col0 + sub_r, mcol = row_base + sub_c;   // transposed block: rows col0.., columns row_base..
            if (mcol < p->Nd) {
#pragma unroll
              for (int it = 0; it < 8; ++it) {
                const int mrow = mrow0 + it * 4;
                if (mrow >= p->Md) break;
                const float* t1 = tile + sub_c * EPI_LD + (it * 4 + sub_r);
                *reinterpret_cast<float4*>(p->D + (long long)mrow * p->ldd + mcol) =
                    make_float4(t1[0], t1[EPI_LD], t1[2 * EPI_LD], t1[3 * EPI_LD]);
              }
            }
          }
        } else if (epi == EPI_ROTATED_ADAM) {
          float* d = p->D + (long long)(row_base + sub_r) * p->ldd + col;      // V~
          float* m2 = p->D2 + (long long)(row_base + sub_r) * p->ldd + col;    // M~
          __nv_bfloat16* xh = p->Dh + (long long)(row_base + sub_r) * p->ldh + col;
          const long long step = 4 * p->ldd, steph = 4 * p->ldh;
          const float b1 = p->beta1, ob1 = 1.0f - p->beta1;
          float4 mm[8], ss[8];
#pragma unroll
          for (int it = 0; it < 8; ++it)
            if (it < n_it) {
              mm[it] = *reinterpret_cast<const float4*>(m2 + it * step);
              ss[it] = *reinterpret_cast<const float4*>(d + it * step);
            }
#pragma unroll
          for (int it = 0; it < 8; ++it)
            if (it < n_it) {
              const float4 g = make_float4(gclip * a[it].x, gclip * a[it].y, gclip * a[it].z, gclip * a[it].w);
              float4 m = mm[it], q = ss[it];
              m.x = b1 * m.x + ob1 * g.x; m.y = b1 * m.y + ob1 * g.y;
              m.z = b1 * m.z + ob1 * g.z; m.w = b1 * m.w + ob1 * g.w;
              q.x = fmaf(beta, q.x, alpha * g.x * g.x); q.y = fmaf(beta, q.y, alpha * g.y * g.y);
              q.z = fmaf(beta, q.z, alpha * g.z * g.z); q.w = fmaf(beta, q.w, alpha * g.w * g.w);
              *reinterpret_cast<float4*>(m2 + it * step) = m;
              *reinterpret_cast<float4*>(d + it * step) = q;
              uint2 o;
              o.x = pack2_bf16(m.x / sqrtf(q.x + eps), m.y / sqrtf(q.y + eps));
              o.y = pack2_bf16(m.z / sqrtf(q.z + eps), m.w / sqrtf(q.w + eps));
              *reinterpret_cast<uint2*>(xh + it * steph) = o;
            }
        } else if (epi == EPI_SECOND_MOMENT) {
          float* d = p->D + (long long)(row_base + sub_r) * p->ldd + col;
          const long long step = 4 * p->ldd;
          float4 ss[8];
#pragma unroll
          for (int it = 0; it < 8; ++it)
            if (it < n_it) ss[it] = *reinterpret_cast<const float4*>(d + it * step);
#pragma unroll
          for (int it = 0; it < 8; ++it)
            if (it < n_it) {
              const float4 g = a[it];
              float4 q = ss[it];
              q.x = fmaf(beta, q.x, alpha * g.x * g.x); q.y = fmaf(beta, q.y, alpha * g.y * g.y);
              q.z = fmaf(beta, q.z, alpha * g.z * g.z); q.w = fmaf(beta, q.w, alpha * g.w * g.w);
              *reinterpret_cast<float4*>(d + it * step) = q;
            }
        } else if (epi == EPI_SCALE_BF16) {
          const float* d = p->D + (long long)(row_base + sub_r) * p->ldd + col;
          __nv_bfloat16* xh = p->Dh + (long long)(row_base + sub_r) * p->ldh + col;
          const long long step = 4 * p->ldd, steph = 4 * p->ldh;
          float4 ss[8];
#pragma unroll
          for (int it = 0; it < 8; ++it)
            if (it < n_it) ss[it] = *reinterpret_cast<const float4*>(d + it * step);
#pragma unroll
          for (int it = 0; it < 8; ++it)
            if (it < n_it) {
              const float4 g = a[it], q = ss[it];
              uint2 o;
              o.x = pack2_bf16(g.x / sqrtf(q.x + eps), g.y / sqrtf(q.y + eps));
              o.y = pack2_bf16(g.z / sqrtf(q.z + eps), g.w / sqrtf(q.w + eps));
              *reinterpret_cast<uint2*>(xh + it * steph) = o;
            }
        } else {  // EPI_SPLIT_BF16
          __nv_bfloat16* dh = p->Dh + (long long)(row_base + sub_r) * p->ldh + col;
          __nv_bfloat16* dl = p->Dl ? p->Dl + (long long)(row_base + sub_r) * p->ldh + col : nullptr;
          const long long steph = 4 * p->ldh;
#pragma unroll
          for (int it = 0; it < 8; ++it)
            if (it < n_it) {
              const float4 g = a[it];
              const float h0 = __bfloat162float(__float2bfloat16_rn(g.x)), h1 = __bfloat162float(__float2bfloat16_rn(g.y));
              const float h2 = __bfloat162float(__float2bfloat16_rn(g.z)), h3 = __bfloat162float(__float2bfloat16_rn(g.w));
              uint2 o;
              o.x = pack2_bf16(h0, h1); o.y = pack2_bf16(h2, h3);
              *reinterpret_cast<uint2*>(dh + it * steph) = o;
              if (dl) {
                uint2 l;
                l.x = pack2_bf16(g.x - h0, g.y - h1); l.y = pack2_bf16(g.z - h2, g.w - h3);
                *reinterpret_cast<uint2*>(dl + it * steph) = l;
              }
            }
        }
        __syncwarp();                             // the tile is rewritten by the next block
      }
      // all tcgen05.ld of this warp have completed (wait::ld): hand the accumulator back
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0)); else mbar_arrive(tempty_bar(acc));
      }
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
  }

  // teardown: every role has left its loop (all waits are bounded)
  // (paired form: neither CTA frees its tensor memory or exits while the other may still signal it)
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_barrier();
  if (warp == 1) {
    tc_fence_after();
    if (PAIR)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// One warp waits, with the kernel's own bounded wait, on an mbarrier that nothing ever arrives on: the
// wait must give up after limit_ns, leave BR_ERR_TIMEOUT in the status word and return.
__global__ void __launch_bounds__(32) k_wait_probe(uint64_t limit_ns, int* status) {
  __shared__ alignas(8) uint64_t bar;
  __shared__ int abort_word;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_word = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0u, &abort_word, status, limit_ns);
}

// ---------------------------------------------------------------------------------------------
// Host side: tensor-map encoding and plans
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// rows = extent of the M / N index, K = contraction extent.
bool encode_operand(CUtensorMap* map, const TcOperand& op, int64_t rows, int64_t K, int box_rows,
                    std::string* err) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) { *err = "cuTensorMapEncodeTiled is not available from the driver"; return false; }
  const int64_t inner = op.mn_major ? rows : K;
  const int64_t outer = op.mn_major ? K : rows;
  const int slots = op.ring_slots > 0 ? op.ring_slots : 1;
  const uint64_t slot_stride = op.ring_slots > 0 ? (uint64_t)op.slot_stride_bytes
                                                 : (uint64_t)op.ld * 2ull * (uint64_t)outer;
  if ((reinterpret_cast<uintptr_t>(op.ptr) & 15) || (op.ld % 8) || (slot_stride % 16)) {
    *err = "tensor-core operand is not 16-byte aligned (pointer, leading dimension or slot stride)";
    return false;
  }
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)outer, (cuuint64_t)slots};
  cuuint64_t strides[2] = {(cuuint64_t)op.ld * 2ull, (cuuint64_t)slot_stride};
  cuuint32_t box[3] = {64u, (cuuint32_t)(op.mn_major ? BK : box_rows), 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(op.ptr), dims, strides, box,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    *err = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r);
    return false;
  }
  return true;
}

typedef void (*TcKernel)(const DevProblem*, int, int, int, long long, int, float, float, int*);
TcKernel kernel_of(bool shared, bool pair, bool fold = false) {
  if (fold) return pair ? k_tc_gemm<false, true, true> : k_tc_gemm<false, false, true>;
  if (pair) return shared ? k_tc_gemm<true, true> : k_tc_gemm<false, true>;
  return shared ? k_tc_gemm<true, false> : k_tc_gemm<false, false>;
}

// Number of CTA pairs (clusters of two) of the paired form that fit on the current device at once;
// 0 when that form is switched off (environment BR_TC_PAIR=0) or cannot be launched.
int pair_capacity(bool shared) {
  static int cap[2] = {-1, -1};
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  int& c = cap[shared ? 1 : 0];
  if (c >= 0) return c;
  c = 0;
  const char* env = std::getenv("BR_TC_PAIR");
  if (env && env[0] == '0') return c;
  TcKernel kernel = kernel_of(shared, true);
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess) {
    cudaGetLastError();
    return c;
  }
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(2u * (unsigned)(sms / 2));
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.attrs = attr; cfg.numAttrs = 1;
  int clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg) != cudaSuccess) { cudaGetLastError(); return c; }
  c = clusters < sms / 2 ? clusters : sms / 2;
  return c;
}

}  // namespace

struct TcPlan {
  bool fold = false;            // launches the folded form (chunked accumulation, running sum in tensor memory)
  bool shared = false;          // launches the shared-operand form of the kernel
  bool pair = false;            // launches the paired form (clusters of two CTAs, 256-row tiles)
  int max_pairs = 0;            // CTA pairs that can be resident at once
  std::vector<int> tile_begin;  // per problem, plus the total at the end
  std::vector<double> prob_flops;
  DevProblem* d_probs = nullptr;
  int n = 0;
  int total_tiles = 0;
  double flops = 0.0;
  int sm_count = 148;
  std::string err;
};

int tc_supported(int device) {
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return 0;
  return prop.major == 10 && get_encode_fn() != nullptr;
}

TcPlan* tc_plan_create(const TcProblem* problems, int n, int device, cudaStream_t s, const char** err) {
  static thread_local std::string last;
  auto fail = [&](const std::string& m) -> TcPlan* { last = m; if (err) *err = last.c_str(); return nullptr; };
  if (n <= 0) return fail("empty plan");
  // The shared-operand form pays off when some problem sums several pairs, and applies when every
  // problem combines at most two distinct A and two distinct B operands.
  auto same_operand = [](const TcOperand& x, const TcOperand& y) {
    return x.ptr == y.ptr && x.ld == y.ld && x.mn_major == y.mn_major && x.ring_slots == y.ring_slots &&
           x.slot_stride_bytes == y.slot_stride_bytes;
  };
  bool shared = false, eligible = true;
  for (int i = 0; i < n; ++i) {
    const TcProblem& q = problems[i];
    if (q.n_pairs < 1 || q.n_pairs > MAX_PAIRS) return fail("tensor-core problem: 1 to 3 operand pairs");
    if (q.n_pairs > 1) shared = true;
    int nA = 0, nB = 0;
    for (int p = 0; p < q.n_pairs; ++p) {
      bool newa = true, newb = true;
      for (int u = 0; u < p; ++u) {
        if (same_operand(q.A[u], q.A[p])) newa = false;
        if (same_operand(q.B[u], q.B[p])) newb = false;
      }
      nA += newa; nB += newb;
    }
    if (nA > 2 || nB > 2) eligible = false;
  }
  shared = shared && eligible;
  // the folded form: every problem asks for it, and none sums several operand pairs
  bool fold = !shared;
  for (int i = 0; i < n; ++i) fold = fold && problems[i].fold_kb > 0 && problems[i].n_pairs == 1;
  if (const char* env = std::getenv("BR_TC_FOLD")) { if (env[0] == '0') fold = false; }      // tuning aid
  int fold_override = 0;
  if (const char* env = std::getenv("BR_TC_FOLD_KB")) { const int v = std::atoi(env); if (v >= 1 && v <= 1024) fold_override = v; }
  const int pairs = pair_capacity(shared);
  const bool pair = pairs > 0;
  const int TM = pair ? 2 * BM : BM;            // rows of a tile
  const int b_box = pair ? BN / 2 : BN;         // rows of B one CTA stages per k-block
  double panel_bytes = kL2PanelBytes;
  if (const char* env = std::getenv("BR_TC_L2_PANEL_MB")) {        // tuning aid
    const double v = std::atof(env);
    if (v >= 1.0 && v <= 512.0) panel_bytes = v * 1e6;
  }
  std::vector<DevProblem> host(n);
  std::vector<int> tile_starts;
  std::vector<double> prob_flops;
  int tile_begin = 0;
  double flops = 0.0;
  for (int i = 0; i < n; ++i) {
    const TcProblem& q = problems[i];
    DevProblem& d = host[i];
    std::memset(&d, 0, sizeof d);
    if (q.n_pairs < 1 || q.n_pairs > MAX_PAIRS || q.Md < 1 || q.Nd < 1 || q.K < 1 ||
        (q.Md % 8) || (q.Nd % 8) || (q.K % 8) || q.Md > (1ll << 30) || q.Nd > (1ll << 30) || q.K > (1ll << 30))
      return fail("tensor-core problem: dimensions must be positive multiples of 8");
    std::string e;
    for (int p = 0; p < q.n_pairs; ++p)
      if (q.A[p].mn_major != q.A[0].mn_major || q.B[p].mn_major != q.B[0].mn_major)
        return fail("tensor-core problem: all pairs must share operand majors");
    if (shared) {
      // distinct operands and the list of products
      int ua[MAX_PAIRS], ub[MAX_PAIRS], nA = 0, nB = 0, combos = 0;
      for (int p = 0; p < q.n_pairs; ++p) {
        int ia = -1, ib = -1;
        for (int u = 0; u < nA; ++u) if (same_operand(q.A[ua[u]], q.A[p])) ia = u;
        for (int u = 0; u < nB; ++u) if (same_operand(q.B[ub[u]], q.B[p])) ib = u;
        if (ia < 0) { ia = nA; ua[nA++] = p; }
        if (ib < 0) { ib = nB; ub[nB++] = p; }
        combos |= (ia | (ib << 1)) << (2 * p);
      }
      for (int u = 0; u < nA; ++u) {
        if (!encode_operand(&d.mapA[u], q.A[ua[u]], q.Md, q.K, BM, &e)) return fail(e);
        if (q.A[ua[u]].ring_slots > 0) { d.a_ring_mask |= 1 << u; d.ring_slots = q.A[ua[u]].ring_slots; }
      }
      for (int u = 0; u < nB; ++u) {
        if (!encode_operand(&d.mapB[u], q.B[ub[u]], q.Nd, q.K, b_box, &e)) return fail(e);
        if (q.B[ub[u]].ring_slots > 0) { d.b_ring_mask |= 1 << u; d.ring_slots = q.B[ub[u]].ring_slots; }
      }
      d.nA = nA; d.nB = nB; d.combos = combos | (q.n_pairs << 8);
    } else {
      for (int p = 0; p < q.n_pairs; ++p) {
        if (!encode_operand(&d.mapA[p], q.A[p], q.Md, q.K, BM, &e)) return fail(e);
        if (!encode_operand(&d.mapB[p], q.B[p], q.Nd, q.K, b_box, &e)) return fail(e);
        if (q.A[p].ring_slots > 0) { d.a_ring_mask |= 1 << p; d.ring_slots = q.A[p].ring_slots; }
        if (q.B[p].ring_slots > 0) { d.b_ring_mask |= 1 << p; d.ring_slots = q.B[p].ring_slots; }
      }
    }
    d.Md = (int32_t)q.Md; d.Nd = (int32_t)q.Nd; d.K = (int32_t)q.K; d.n_pairs = q.n_pairs;
    d.a_mn = q.A[0].mn_major; d.b_mn = q.B[0].mn_major; d.epilogue = q.epilogue;
    d.tiles_m = (int32_t)((q.Md + TM - 1) / TM);
    d.tiles_n = (int32_t)((q.Nd + BN - 1) / BN);
    d.tile_begin = tile_begin;
    d.tile_count = d.tiles_m * d.tiles_n;
    // A symmetric product on square tiles lists only the tiles of the upper triangle, so that the
    // round-robin walk gives every CTA pair the same number of computed tiles.
    d.tri = (q.symmetric && TM == BN && d.tiles_m == d.tiles_n) ? 1 : 0;
    if (d.tri) d.tile_count = d.tiles_m * (d.tiles_m + 1) / 2;
    {
      // Estimated DRAM reads of the two walks: the resident panel's operand once, the other once per
      // group.  Group = as many blocks as keep the panel within its share of L2.
      int nA = 0, nB = 0;
      for (int p = 0; p < q.n_pairs; ++p) {
        bool newa = true, newb = true;
        for (int u = 0; u < p; ++u) {
          if (same_operand(q.A[u], q.A[p])) newa = false;
          if (same_operand(q.B[u], q.B[p])) newb = false;
        }
        nA += newa; nB += newb;
      }
      const double stripeA = (double)TM * (double)q.K * 2.0 * nA, stripeB = (double)BN * (double)q.K * 2.0 * nB;
      const double totalA = stripeA * d.tiles_m, totalB = stripeB * d.tiles_n;
      auto clampi = [](double v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : (int)v); };
      const int gM = clampi(panel_bytes / stripeA, 1, d.tiles_m), gN = clampi(panel_bytes / stripeB, 1, d.tiles_n);
      const double trafficM = totalA + totalB * ((d.tiles_m + gM - 1) / gM);
      const double trafficN = totalB + totalA * ((d.tiles_n + gN - 1) / gN);
      d.raster_n = trafficN < trafficM ? 1 : 0;
      d.group = d.raster_n ? gN : gM;
    }
    tile_starts.push_back(tile_begin);
    tile_begin += d.tile_count;
    d.tau_max = q.tau_max;
    d.dyn_scalars = q.dyn_scalars;
    d.alpha = q.alpha; d.beta = q.beta; d.eps = q.eps; d.beta1 = q.beta1;
    d.symmetric = q.symmetric ? 1 : 0;
    d.clip = q.clip_mode ? q.clip : nullptr; d.clip_slots = q.clip_slots; d.clip_mode = q.clip_mode;
    d.fold_kb = fold ? (fold_override ? fold_override : q.fold_kb) : 0;
    if (d.clip && (q.clip_slots < 1 || (q.clip_mode == 1 && q.epilogue != EPI_ROTATED_ADAM) ||
                   (q.clip_mode == 2 && q.epilogue != EPI_AXPBY_F32)))
      return fail("tensor-core problem: clipping applies to the rotated-Adam and factor epilogues");
    if (q.symmetric && (q.Md != q.Nd || q.epilogue != EPI_AXPBY_F32))
      return fail("tensor-core problem: a symmetric product needs a square fp32 result");
    d.D = q.D; d.ldd = q.ldd; d.Dh = q.Dh; d.Dl = q.Dl; d.ldh = q.ldh; d.D2 = q.D2;
    const bool need_D = q.epilogue != EPI_SPLIT_BF16;
    const bool need_H = q.epilogue == EPI_SPLIT_BF16 || q.epilogue == EPI_SCALE_BF16 || q.epilogue == EPI_ROTATED_ADAM;
    if (q.epilogue == EPI_ROTATED_ADAM && (!q.D2 || (reinterpret_cast<uintptr_t>(q.D2) & 15)))
      return fail("tensor-core problem: second in/out pointer missing or misaligned");
    if ((need_D && (!q.D || (q.ldd % 4) || (reinterpret_cast<uintptr_t>(q.D) & 15))) ||
        (need_H && (!q.Dh || (q.ldh % 8) || (reinterpret_cast<uintptr_t>(q.Dh) & 15))) ||
        (q.Dl && (reinterpret_cast<uintptr_t>(q.Dl) & 15)))
      return fail("tensor-core problem: output pointer missing or misaligned");
    const double flops_before = flops;
    if (q.symmetric) {
      // executed work: the tiles that touch the upper triangle
      int64_t computed = 0;
      for (int64_t rb = 0; rb < d.tiles_m; ++rb)
        for (int64_t cb = 0; cb < d.tiles_n; ++cb)
          if (rb * TM < cb * BN + BN) ++computed;
      flops += 2.0 * (double)computed * TM * BN * (double)q.K * q.n_pairs;
    } else {
      flops += 2.0 * (double)q.Md * (double)q.Nd * (double)q.K * q.n_pairs;
    }
    prob_flops.push_back(flops - flops_before);
  }
  TcPlan* plan = new TcPlan();
  plan->fold = fold;
  plan->shared = shared;
  plan->pair = pair;
  plan->max_pairs = pairs;
  tile_starts.push_back(tile_begin);
  plan->tile_begin = tile_starts;
  plan->prob_flops = prob_flops;
  plan->n = n;
  plan->total_tiles = tile_begin;
  plan->flops = flops;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) == cudaSuccess) plan->sm_count = prop.multiProcessorCount;
  cudaError_t ce = cudaMalloc(&plan->d_probs, sizeof(DevProblem) * n);
  if (ce == cudaSuccess)
    ce = cudaMemcpyAsync(plan->d_probs, host.data(), sizeof(DevProblem) * n, cudaMemcpyHostToDevice, s);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(s);   // `host` goes out of scope
  if (ce != cudaSuccess) {
    if (plan->d_probs) cudaFree(plan->d_probs);
    delete plan;
    return fail(std::string("plan upload: ") + cudaGetErrorString(ce));
  }
  return plan;
}

void tc_plan_destroy(TcPlan* p) {
  if (!p) return;
  if (p->d_probs) cudaFree(p->d_probs);
  delete p;
}

double tc_plan_flops(const TcPlan* p) { return p ? p->flops : 0.0; }

cudaError_t tc_plan_launch_range(TcPlan* p, int first, int count, long long calls, int tau, float dyn_alpha,
                                 float dyn_beta, int* status_word, cudaStream_t s) {
  if (first < 0 || count < 1 || first + count > p->n) return cudaErrorInvalidValue;
  const int t0 = p->tile_begin[first], t1 = p->tile_begin[first + count];
  const int tiles = t1 - t0;
  TcKernel kernel = kernel_of(p->shared, p->pair, p->fold);
  // per-device attribute: set again when another device is current (cheap, idempotent)
  const int smem_bytes = p->fold ? SMEM_BYTES_FOLD : SMEM_BYTES;
  cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  if (p->pair) {
    const int units = tiles < p->max_pairs ? tiles : p->max_pairs;
    cfg.gridDim = dim3(2u * (unsigned)units);
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
  } else {
    cfg.gridDim = dim3((unsigned)(tiles < p->sm_count ? tiles : p->sm_count));
  }
  cfg.blockDim = dim3(p->fold ? FOLD_THREADS : NUM_THREADS);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = s;
  return cudaLaunchKernelEx(&cfg, kernel, (const DevProblem*)p->d_probs, p->n, t0, t1, calls, tau, dyn_alpha,
                            dyn_beta, status_word);
}

cudaError_t tc_plan_launch(TcPlan* p, long long calls, int tau, float dyn_alpha, float dyn_beta,
                           int* status_word, cudaStream_t s) {
  return tc_plan_launch_range(p, 0, p->n, calls, tau, dyn_alpha, dyn_beta, status_word, s);
}

cudaError_t tc_wait_probe(uint64_t limit_ns, int* status_word, cudaStream_t s) {
  k_wait_probe<<<1, 32, 0, s>>>(limit_ns, status_word);
  return cudaGetLastError();
}

double tc_plan_flops_range(const TcPlan* p, int first, int count) {
  double f = 0.0;
  for (int i = first; i < first + count && i < p->n; ++i) f += p->prob_flops[i];
  return f;
}

}  // namespace br
