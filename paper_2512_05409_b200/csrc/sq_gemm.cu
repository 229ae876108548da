// Hybrid SQ-format GEMM on the sm_100a tensor cores (tcgen05, kind::i8).
//
//   acc[m,n] = sum_j ( (dq4[m,j] << e[m]) + [j in S_m] vals[m,j] ) * code[n,j]
//   out[m,n] = bf16( ((float)acc * s_hi[m]) * s_w[n] )
//
// sm_100 has no INT4 MMA, so both operands are widened to 8 bits on chip.  The two
// components of the activation live on one integer grid (the dense one coarsened by
// 2^e), so they go into ONE int32 accumulator in tensor memory:
//   dynamic positions: the k sparse INT8 entries of every bank overwrite the (zero) places
//     they belong to in the widened dense tile before the tensor core sees it;
//   static positions (Section 3.3, Fig. 2b: the mask only selects and gathers activation
//     tiles because the weight rows were reordered offline): vals [M, G*k] and w_sparse
//     [N, G*k] are plain INT8 matrices, so the sparse product is G*k/128 extra K steps whose
//     tiles TMA writes straight into the same shared-memory stages (swizzled by the TMA
//     unit, no thread touches them) and whose MMAs accumulate into the same tile.
//
// Operand encodings inside the kernel (chosen so the widening is a few logic ops on
// eight nibbles at a time, never a per-byte sign extension):
//   A is fed UNSIGNED with an offset of 128:  a_u = a + 128, a in [-127, 127].
//     dense:  nibble q in two's complement -> u = q ^ 8 = q + 8 in [1, 15];
//             a_u = u * 2^e + (128 - 8 * 2^e)      (no carries between bytes)
//     sparse (merged): a_u = vals ^ 0x80;  sparse (extra K steps): A signed, vals as stored
//   B is fed SIGNED as 16 * code: a nibble moved to the top of its byte (w_sparse is stored
//   that way already).
//   Hence acc_internal = 16 * acc + 2048 * colsum[n]; the epilogue undoes both exactly.
//   |acc_internal| <= K * 255 * 112 < 2^31 for K <= 65536.
//
// K order inside a 32-element MMA block: eight nibbles come out of one 32-bit word as
// the four even elements and the four odd ones, so both operands store a block as
// [16 even elements | 16 odd elements].  The contraction does not care as long as A
// and B agree.
//
// Shared-memory operand layout: K-major, 128-byte rows (one K step = 128 elements),
// 128-byte swizzle (the 16-byte chunk index is XORed with row % 8), 8-row groups 1024
// bytes apart: the canonical layout a tcgen05 shared-memory descriptor describes.
//
// Tiling: a CTA accumulates 256 rows x 256 output channels as two 128-row sub-tiles that share
// every widened weight stage and fill all 512 tensor-memory columns.  Above 128 rows the CTAs
// work in PAIRS (clusters of two, `tcgen05.mma.cta_group::2`): the pair computes 512 x 256, each
// CTA owns 256 rows of A and only HALF of the weight tile, which the pair's tensor cores read
// from both shared memories.  Per MMA a CTA then widens a quarter less and its shared memory
// serves a third less operand traffic; shared-memory bandwidth (widening stores + tensor-core
// operand reads) is what bounds the single-CTA form.  The last, partial wave of a launch is cut
// into tiles of one sub-tile per CTA so that it spreads over twice as many SMs.
//
// Kernel organisation: persistent, one CTA per SM, warp-specialised, two-level pipeline
// (packed ring -> widened ring -> tensor cores).  In a pair only the leader CTA's MMA thread
// issues; both CTAs' producers arrive on the leader's "full" barriers (remote mbarrier
// arrives), and the MMA completions are multicast to both CTAs' "empty" barriers.
//   warp  13    one thread streams the packed 4-bit tiles (256 rows x 64 B of A, 256 or 128 rows
//               of B per K step) into a ring of NP packed stages by TMA
//   warps 0-7   producers: read their chunks of a packed stage, widen them, store the
//               swizzled 8-bit layout into a ring of NS widened stages; dynamic positions with
//               16 sparse entries per row and K step: each thread then merges the sparse INT8
//               entries of one of the 32 rows its warp has just written (byte stores, four
//               positions per SWAR step)
//   warps 9-12  for every tile: epilogue (tcgen05.ld, dequantise, bf16, 16-byte stores);
//               dynamic positions in the other formats: they do the merge, between the
//               producers and the MMA thread
//   warp  8     one thread issues the MMAs and commits stage / accumulator barriers
//   warp  14    static positions: one thread issues the TMA loads of the sparse K steps
// Every wait is bounded; a wait that runs out raises an abort flag that releases all
// other waits, the kernel records SQ_ERR_TIMEOUT and frees its tensor memory.
//
// Few rows (at most 128): a launch has only N/256 tiles, so given a workspace K is cut into
// parts (work item = column tile x part of K) whose raw partial sums a second kernel adds.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <string.h>

#include "sq_device.cuh"

#include "sq_host.h"

// How the producers wait for a packed stage to land / a widened stage to be consumed: parked by
// the hardware (idle producers must not take issue slots from the epilogue warps); the TMA
// threads (one lane each) poll.
#define WAIT_PE mbar_wait_park
#define WAIT_PF mbar_wait_park
#define WAIT_T mbar_wait
namespace sq {

namespace {

constexpr int BM = 128;   // rows of one sub-tile = TMEM lanes
constexpr int BN = 256;   // output channels per tile = TMEM columns of one accumulator
constexpr int BK = 128;   // K elements per pipeline step = bytes per operand row
constexpr int kProdWarps = 8;
constexpr int kProdThreads = kProdWarps * 32;
constexpr int kMmaWarp = kProdWarps;
constexpr int kEpiWarps = 4;
// Letting the (by then idle) producer warps read out two thirds of a tile's accumulators was
// measured slower than leaving the epilogue to its own four warps (the producers then refill
// the pipeline later), so it is compiled out; the hand-shake below supports both.
constexpr bool kProducersJoinEpilogue = false;
constexpr int kEpiHelpers = kEpiWarps + (kProducersJoinEpilogue ? kProdWarps : 0);
constexpr int kEpiStride = kProducersJoinEpilogue ? 3 : 1;  // warps per TMEM lane quarter
constexpr int kTmaWarp = kProdWarps + 1 + kEpiWarps;  // packed dense tiles
constexpr int kTmaSparseWarp = kTmaWarp + 1;          // INT8 tiles of the sparse K steps
constexpr int kMma2Warp = kTmaSparseWarp + 1;           // second MMA issuer (pre-widened activations)
constexpr int kThreads = (kProdWarps + 1 + kEpiWarps + 3) * 32;
// Pre-widened activations: the epilogue is what the tensor pipe waits for between tiles and one
// warp per scheduler leaves its latencies (tensor-memory load, staging, TMA hand-over) exposed,
// so four more warps (16..19) join it: two warps per tensor-memory lane quarter.
constexpr int kEpiWarpsA8 = 8;
constexpr int kThreadsA8 = kThreads + (kEpiWarpsA8 - kEpiWarps) * 32;
constexpr int kCtlBytes = 256;            // barriers, tensor-memory slot, abort flag
constexpr int kEpiConstBytes = 2 * BN * 4;  // per tile: 2048 * colsum[n] and s_w[n] of its columns
constexpr int kOutBlock = 32 * 32 * 2;        // one staged output block: 32 rows x 32 bf16
constexpr int kModeMergeEpi = 0, kModeTma = 1, kModeMergeProd = 2, kModeA8 = 3, kModeIndep = 4;  // see gemm_kernel
constexpr int threads_of(int mode) { return mode == kModeA8 ? kThreadsA8 : kThreads; }
constexpr int kRowsPerWarp = 2 * BM / kProdWarps;  // rows of A a producer warp widens per stage
constexpr int kATasks = kRowsPerWarp / 8;  // 16-byte packed chunks of A per producer thread per step

// What depends on how many CTAs share a tensor-core tile.  PAIR = 1: one CTA computes 256 x 256
// alone.  PAIR = 2: the two CTAs of a cluster compute 512 x 256 with `cta_group::2` MMAs; each
// owns 256 rows of A and HALF of the weight tile (128 output channels), which the pair's tensor
// cores read from both shared memories, so a CTA widens and holds a quarter less per MMA and
// its shared memory serves a third less operand traffic -- the pipe this kernel is bound by.
template <int PAIR, int MODE = kModeTma>
struct Geo {
  // rows of A per stage: two sub-tiles per CTA of a pair; a lone CTA (at most 128 rows in the
  // whole launch) only ever has one, and the room goes to a third widened stage
  static constexpr int kRowsA = PAIR == 1 ? BM : 2 * BM;
  static constexpr int kStageA = kRowsA * BK;  // 16 / 32 KB widened
  // packed A per stage: 64 bytes per row; none when TMA delivers 8-bit activations
  static constexpr int kPackA = MODE == kModeA8 ? 0 : kRowsA * (BK / 2);
  // stages of widened (8-bit) operands; 8-bit activation tiles land there directly, so that ring
  // alone hides their latency and gets the room the packed A ring does not need
  static constexpr int NS = PAIR == 2 ? (MODE == kModeA8 ? 4 : 3) : 3;
  // stages of packed (4-bit) operands as TMA delivers them (with 8-bit activations only weights
  // pass through them, and the third stage's room goes to the output staging below)
  static constexpr int NP = MODE == kModeA8 ? 2 : 3;
  static constexpr int BNL = BN / PAIR;          // weight rows (output channels) held by one CTA
  static constexpr int kStageB = BNL * BK;       // 32 / 16 KB
  static constexpr int kPackB = BNL * (BK / 2);  // 16 / 8 KB
  static constexpr int kRowsPerWarpB = BNL / kProdWarps;
  static constexpr int kBTasks = kRowsPerWarpB / 8;
  // output staging (8-bit activation mode): a 32-row x 32-column bf16 block per epilogue warp,
  // which leave through TMA stores instead of one 16-byte store per thread and row
  static constexpr int kOutStage = MODE == kModeA8 ? kEpiWarpsA8 * kOutBlock : 0;
  static constexpr int kSmemBytes =
      NS * (kStageA + kStageB) + NP * (kPackA + kPackB) + kOutStage + kCtlBytes + kEpiConstBytes;
};
constexpr int kMergeTasks = 8;  // sparse 4-entry words per merge thread per stage kept in registers

struct GemmParams {
  const uint8_t* dq4;
  const int8_t* vals;
  const uint8_t* idx;  // dynamic positions [M,G,k] or nullptr
  const uint8_t* pos;  // static positions [G,k] or nullptr
  const float* s_hi;
  const float* s_lo;  // independent scales only
  const uint8_t* shift;
  const uint8_t* wq4;
  const float* s_w;
  const int32_t* colsum;
  uint16_t* out;
  int32_t* acc_out;
  int* status;
  int32_t* ws;     // split-K: raw partial accumulators [splits][M][N]; nullptr: the parts of a tile form a
                   // thread-block cluster and add their partial sums through distributed shared memory
  int M, N, K, b, k;
  int log2k;       // log2(k) when the word path is usable, else -1
  int SS;          // sparse K steps per tile (static positions through TMA), else 0
  int splits;      // split-K: work items per output tile (each walks KS dense K steps), else 1
  int KS;          // dense K steps per work item
  // work list: `n_pairs` tiles of two sub-tiles per CTA followed by `n_singles` tiles of one;
  // a row unit is 128 rows per CTA of the pair (128 or 256 rows)
  int n_pairs, n_singles, n_split;  // n_split: singles that come from cutting pair tiles in two
  int mp, mu, tiles_n;              // row pairs, row units, column tiles
  int rows_a;                       // rows the activation TMA boxes fetch (a lone CTA: M rounded up to 8, so
                                    // that a few tokens do not cost the TMA unit 128 row requests per step)
};

struct Tile {
  int m0, n0, nsub;  // first row of THIS CTA, first output channel of the tile, sub-tiles per CTA
  int nb0;           // first weight row THIS CTA loads and widens
  int split, k0;     // split-K: which part of K this work item covers and its first K step
  int ss;            // sparse K steps of this work item (the first part of K takes them all)
};

// Entry j of the work list (identical in every role of both CTAs of a pair, up to the rank).
template <int PAIR, bool SPLITK>
__device__ __forceinline__ Tile tile_of(const GemmParams& p, int j, int rank) {
  constexpr int U = BM * PAIR;  // rows of a row unit
  Tile t;
  t.split = 0;
  if (j < p.n_pairs) {
    t.m0 = (j % p.mp) * (2 * U);
    t.n0 = (j / p.mp) * BN;
    t.nsub = 2;
  } else {
    const int s = j - p.n_pairs;
    t.nsub = 1;
    if (s < p.n_split) {
      const int pj = p.n_pairs + s / 2;
      t.m0 = (pj % p.mp) * (2 * U) + (s & 1) * U;
      t.n0 = (pj / p.mp) * BN;
    } else {  // the odd last row unit (with split-K: `splits` work items per column tile)
      const int q = s - p.n_split;
      t.m0 = (p.mu - 1) * U;
      if (SPLITK) {  // the parts of a tile are neighbours in the work list (= one cluster, if clustered)
        t.n0 = (q / p.splits) * BN;
        t.split = q % p.splits;
      } else {
        t.n0 = q * BN;
      }
    }
  }
  t.m0 += rank * t.nsub * BM;
  t.nb0 = t.n0 + rank * (BN / PAIR);
  t.k0 = SPLITK ? t.split * p.KS : 0;
  t.ss = (!SPLITK || t.split == 0) ? p.SS : 0;
  return t;
}

// Shared-memory matrix descriptor: K-major, SWIZZLE_128B, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);  // start address
  d |= (uint64_t)1 << 16;                    // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset
  d |= (uint64_t)1 << 46;                    // descriptor version (sm_100)
  d |= (uint64_t)2 << 61;                    // SWIZZLE_128B
  return d;
}

// Instruction descriptor: D = s32, A = u8 or s8, B = s8, both K-major, N = BN.
__device__ __forceinline__ constexpr uint32_t make_idesc(bool a_signed, int m) {
  return (2u << 4)                       // D format: S32
         | ((a_signed ? 1u : 0u) << 7)   // A format: 0 = unsigned, 1 = signed 8-bit
         | (1u << 10)                    // B format: signed 8-bit
         | ((uint32_t)(BN >> 3) << 17)   // N
         | ((uint32_t)(m >> 4) << 24);   // M (of the whole instruction: 128 per participating CTA)
}

// Four bank-local indices in one word -> their K positions inside the bank's 32-blocks
// (even elements first, then odd ones), bytewise.
__device__ __forceinline__ uint32_t kpos4(uint32_t w) {
  return (w & 0x60606060u) | ((w & 0x01010101u) << 4) | ((w >> 1) & 0x0F0F0F0Fu);
}
__device__ __forceinline__ uint32_t kpos1(uint32_t jj) {
  return (jj & 0x60u) | ((jj & 1u) << 4) | ((jj & 31u) >> 1);
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// 2-D tiled TMA load into this CTA's shared memory; x (bytes here) must be a multiple of 16.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}


// 2-D tiled TMA store from this CTA's shared memory (rows and columns past the tensor's extent
// are dropped); x in elements, x * element size a multiple of 16.  One bulk group per store.
__device__ __forceinline__ void tma_store_2d(uint32_t src, const CUtensorMap* map, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map), "r"(x), "r"(y),
               "r"(src)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Wait until all but the newest N of this thread's bulk groups have read their shared memory ...
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
// ... or have completed altogether.
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

}  // namespace

// Arrive on / wait for a barrier that lives in the pair's leader CTA.
template <int PAIR>
__device__ __forceinline__ void arrive_leader(uint32_t bar) {
  if (PAIR == 2) mbar_arrive_cta(bar, 0);
  else mbar_arrive(bar);
}
template <int PAIR>
__device__ __forceinline__ bool wait_leader(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return PAIR == 2 ? mbar_wait_cluster(bar, parity, abort_flag) : mbar_wait(bar, parity, abort_flag);
}

// PAIR: CTAs per tensor-core tile (see Geo).
// MODE: how the sparse part reaches the tensor core.
//   kModeMergeEpi   the epilogue warps merge the sparse entries into every widened A stage
//                   (any bank size and k; also static positions TMA cannot fetch)
//   kModeTma        static positions: TMA-fed extra K steps
//   kModeMergeProd  16 sparse entries per row and K step (k/b = 1/8): every producer thread
//                   merges one row of the 32 its warp has just widened -- no hand-over to
//                   other warps, eight warps share the work
//   kModeIndep      static positions with independent scales: like kModeTma, but the sparse K
//                   steps accumulate into a tensor-memory accumulator of their own (the second
//                   sub-tile's columns: every tile has one sub-tile per CTA) and the epilogue
//                   joins the two integer sums in fp32 with the row's two scales
//   kModeA8         the caller gave a workspace of M*K bytes: expand_a8_kernel has written the
//                   activations there as merged 8-bit operands (dense part widened, sparse
//                   entries in place, K order of the MMA blocks), once per row instead of once
//                   per row AND column tile; TMA brings those tiles straight into the widened
//                   ring and the producers widen only the weights.  No sparse K steps either.
template <int PAIR, int MODE, bool SPLITK>
__global__ void __launch_bounds__(threads_of(MODE), 1)
    gemm_kernel(const GemmParams p, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                const __grid_constant__ CUtensorMap map_a4, const __grid_constant__ CUtensorMap map_b4) {
  using G = Geo<PAIR, MODE>;
  constexpr bool INDEP = MODE == kModeIndep;
  constexpr bool STMA = MODE == kModeTma || INDEP, PMERGE = MODE == kModeMergeProd, A8 = MODE == kModeA8;
  constexpr bool ATMA = STMA || A8;  // the second TMA thread fills (some or all) A stages
  // With 8-bit activations the epilogue is what the tensor pipe waits for between tiles, and its
  // stores (a thread per row: 32 different 128-byte lines per 16-byte store instruction) were
  // most of it.  There the bf16 block is staged in shared memory and written by TMA (map_b,
  // otherwise unused in this mode, describes `out`).
  constexpr bool TSTORE = A8 && !SPLITK;
  constexpr int kEpiAll = A8 ? kEpiWarpsA8 : kEpiHelpers;  // warps that read out a tile
  constexpr int kEpiStep = A8 ? kEpiWarpsA8 / 4 : kEpiStride;  // ... per tensor-memory lane quarter
  constexpr int NS = G::NS, NP = G::NP;
  constexpr int kStageA = G::kStageA, kStageB = G::kStageB, kPackB = G::kPackB, kBTasks = G::kBTasks, kPackA = G::kPackA;
  // The kernel has no static shared memory, so the dynamic block starts at the 1024-byte
  // aligned base the swizzled operand layout needs; checked below, never assumed.
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = smem_raw;
  // (uniform over the pair: both CTAs see the same offset of the dynamic block)
  if ((smem_u32(smem_raw) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicExch(p.status, (int)SQ_ERR_CUDA);
    return;
  }
  uint8_t* sA = smem;                      // NS x [kRowsA][128] widened A
  uint8_t* sB = sA + NS * kStageA;         // NS x [BNL][128] widened B
  uint8_t* sPA = sB + NS * kStageB;        // NP x [256][64]  packed A as loaded
  uint8_t* sPB = sPA + NP * kPackA;        // NP x [BNL][64]  packed B as loaded
  uint8_t* sOut = sPB + NP * kPackB;       // kEpiWarpsA8 x [32][64] staged output blocks (TSTORE)
  uint8_t* sCtl = sOut + G::kOutStage;
  // mbarriers.  "leader" = waited for by the MMA thread of the pair's rank-0 CTA only; both
  // CTAs arrive there.  Everything else is local to a CTA (signalled in both by multicast
  // commits where the tensor core is the one that arrives).
  const uint32_t bar_full = smem_u32(sCtl);         // NS, leader: dense K step widened (and merged)
  const uint32_t bar_empty = bar_full + 8 * NS;     // NS: widened stage consumed by the MMAs
  const uint32_t bar_sfull = bar_empty + 8 * NS;    // NS: sparse K step filled by this CTA's TMA
  const uint32_t bar_pfull = bar_sfull + 8 * NS;    // NP: packed stage landed
  const uint32_t bar_pempty = bar_pfull + 8 * NP;   // NP: packed stage read into registers
  const uint32_t bar_tfull = bar_pempty + 8 * NP;   // accumulators complete
  const uint32_t bar_tempty = bar_tfull + 8;        // leader: accumulators read out
  const uint32_t bar_wfull = bar_tempty + 8;        // NS: dense K step widened, sparse entries not merged yet
  const uint32_t bar_eready = bar_wfull + 8 * NS;   // epilogue: column constants staged, every helper present
  const uint32_t bar_edone = bar_eready + 8;        // epilogue: every helper done with the constants
  const uint32_t bar_sfullp = bar_edone + 8;        // NS, leader: sparse K step filled by the peer's TMA
  // leader, two issuing threads: the SECOND sub-tile's accumulator read out (bar_tempty is then the
  // first one's alone, so its thread starts the next tile while the second is still being drained)
  const uint32_t bar_tempty1 = bar_sfullp + 8 * NS;
  static_assert(8 * (5 * NS + 2 * NP + 5) + 16 <= kCtlBytes, "control block too small");
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sCtl + 8 * (5 * NS + 2 * NP + 5));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sCtl + 8 * (5 * NS + 2 * NP + 5) + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // Rank in the pair (0 = leader; clusters are (PAIR,1,1), so it is blockIdx.x % PAIR), this
  // pair's index and the number of pairs.  Spelled out at every use instead of being kept in
  // variables: derived from blockIdx/gridDim right where they are needed they stay in the
  // uniform datapath, which the single-thread roles (MMA issue, TMA) depend on.
#define rank ((int)blockIdx.x % PAIR)
#define cl ((int)blockIdx.x / PAIR)
#define ncl ((int)gridDim.x / PAIR)
  const int KS = SPLITK ? p.KS : p.K / BK;  // dense K steps of a work item (all of K unless split)
  const int nwork = p.n_pairs + p.n_singles;

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      // Every thread arrives for itself right after its own proxy fence (one arrival per warp
      // behind a __syncwarp was measured slower).  Static positions: the producers complete a
      // dense stage; otherwise the merge warps do.
      // (TMA-delivered activations: plus, per CTA of the pair, the arrival that announces its tile)
      mbar_init(bar_full + 8 * s, PAIR * ((STMA || PMERGE || A8) ? kProdWarps : kEpiWarps) * 32 + (A8 ? PAIR : 0));
      mbar_init(bar_wfull + 8 * s, kProdWarps * 32);
      mbar_init(bar_empty + 8 * s, A8 ? 2 : 1);  // one commit per MMA-issuing thread
      mbar_init(bar_sfull + 8 * s, 1);
      mbar_init(bar_sfullp + 8 * s, 1);
    }
    for (int s = 0; s < NP; ++s) {
      mbar_init(bar_pfull + 8 * s, 1);
      mbar_init(bar_pempty + 8 * s, kProdThreads);
    }
    mbar_init(bar_tfull, A8 ? 2 : 1);
    mbar_init(bar_tempty, PAIR * kEpiAll * 32);
    mbar_init(bar_tempty1, PAIR * kEpiAll * 32);
    mbar_init(bar_eready, kEpiAll * 32);
    mbar_init(bar_edone, kEpiAll * 32);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kMmaWarp) {
    tmem_alloc<PAIR>(smem_u32(tmem_slot), 2 * BN);
    tmem_relinquish<PAIR>();
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR == 2) cluster_sync_all();  // the peer's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // ---- epilogue of one tile, shared by the epilogue warps and the producers (which have run
  //      out of free stages by the time a tile completes): warp w reads TMEM lane quarter
  //      w % 4; the three warps of a quarter split the tile's 32-column chunks.
  int32_t* s_cs = reinterpret_cast<int32_t*>(sCtl + kCtlBytes);  // 2048 * colsum of the tile's columns
  float* s_sw = reinterpret_cast<float*>(sCtl + kCtlBytes + BN * 4);
  uint32_t oc = 0;  // TSTORE: blocks this warp has staged so far
  auto epilogue_share = [&](const Tile& t, uint32_t tile_count, int helper) -> bool {
    const int q = warp & 3;
    // this thread's two rows' scales, requested before the wait so that no chunk waits for them
    float sh2[2];
#pragma unroll
    for (int sub = 0; sub < 2; ++sub) {
      const int m = t.m0 + sub * BM + 32 * q + lane;
      sh2[sub] = (sub < t.nsub && m < p.M) ? __ldg(p.s_hi + m) : 0.f;
    }
    float sl = 0.f;  // independent scales: the row's dense scale (one sub-tile per CTA)
    if (INDEP) {
      const int m = t.m0 + 32 * q + lane;
      sl = m < p.M ? __ldg(p.s_lo + m) : 0.f;
    }
    if (!mbar_wait_idle(bar_tfull, tile_count & 1u, abort_flag)) return false;
    tc_fence_after();
    mbar_arrive(bar_eready);
    if (!mbar_wait(bar_eready, tile_count & 1u, abort_flag)) return false;
    bool released0 = false;
    for (int ci = helper; ci < t.nsub * (BN / 32); ci += kEpiStep) {
      const int sub = ci / (BN / 32), c0 = (ci % (BN / 32)) * 32;
      if (A8 && sub == 1 && !released0) {  // this thread's loads of the first accumulator are complete
        tc_fence_before();
        arrive_leader<PAIR>(bar_tempty);
        released0 = true;
      }
      const int m = t.m0 + sub * BM + 32 * q + lane;
      const float sh = sub == 0 ? sh2[0] : sh2[1];
      uint32_t v[32];
      uint32_t vs[INDEP ? 32 : 1];  // independent scales: the sparse product's accumulators
      tmem_ld32(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(sub * BN + c0), v);
      if constexpr (INDEP) tmem_ld32(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(BN + c0), vs);
      tmem_ld_wait();
      const int n0 = t.n0 + c0;
      if constexpr (INDEP) {
        // out = bf16(fmaf(acc_hi, s_hi, acc_lo * s_lo) * s_w): the dense sum carries the unsigned
        // operand's offset (2048 * colsum) and both sums the weights' factor 16
        if (m < p.M && n0 < p.N) {
#pragma unroll
          for (int c8 = 0; c8 < 32; c8 += 8) {
            if (n0 + c8 < p.N) {
              int lo[8], hi[8];
              uint32_t o[4];
#pragma unroll
              for (int cc = 0; cc < 8; ++cc) {
                lo[cc] = ((int)v[c8 + cc] - s_cs[c0 + c8 + cc]) >> 4;
                hi[cc] = (int)vs[c8 + cc] >> 4;
              }
#pragma unroll
              for (int cc = 0; cc < 8; cc += 2) {
                const float f0 = __fmul_rn(__fmaf_rn((float)hi[cc], sh, __fmul_rn((float)lo[cc], sl)), s_sw[c0 + c8 + cc]);
                const float f1 = __fmul_rn(__fmaf_rn((float)hi[cc + 1], sh, __fmul_rn((float)lo[cc + 1], sl)), s_sw[c0 + c8 + cc + 1]);
                o[cc >> 1] = pack_bf16x2(f0, f1);
              }
              *reinterpret_cast<uint4*>(p.out + (size_t)m * p.N + n0 + c8) = make_uint4(o[0], o[1], o[2], o[3]);
              if (p.acc_out != nullptr) {  // [2, M, N]: dense sums, then sparse sums
                int4* dst = reinterpret_cast<int4*>(p.acc_out + (size_t)m * p.N + n0 + c8);
                dst[0] = make_int4(lo[0], lo[1], lo[2], lo[3]);
                dst[1] = make_int4(lo[4], lo[5], lo[6], lo[7]);
                dst = reinterpret_cast<int4*>(p.acc_out + (size_t)p.M * p.N + (size_t)m * p.N + n0 + c8);
                dst[0] = make_int4(hi[0], hi[1], hi[2], hi[3]);
                dst[1] = make_int4(hi[4], hi[5], hi[6], hi[7]);
              }
            }
          }
        }
      } else if (SPLITK && p.ws == nullptr) {
        // clustered split-K: this CTA's raw partial sums go to its own shared memory (the operand
        // rings are idle by now: a CTA has a single work item), row-major [128][256] int32 with
        // the 16-byte chunks of a row XOR-swizzled by the row so that a warp's stores (one row
        // per lane) spread over the banks; the cluster adds them at the end of the kernel
        if (m < p.M) {
          const int r = 32 * q + lane;
          uint8_t* prow = smem + (size_t)r * (BN * 4);
#pragma unroll
          for (int c4 = 0; c4 < 8; ++c4)
            *reinterpret_cast<int4*>(prow + ((((c0 >> 2) + c4) ^ (r & 7)) << 4)) =
                make_int4((int)v[4 * c4], (int)v[4 * c4 + 1], (int)v[4 * c4 + 2], (int)v[4 * c4 + 3]);
        }
      } else if (SPLITK) {
        // split-K: this work item's raw partial sums; splitk_finish_kernel adds the parts
        if (m < p.M) {
          int32_t* wrow = p.ws + ((size_t)t.split * p.M + m) * p.N + n0;
          for (int c8 = 0; c8 < 32 && n0 + c8 < p.N; c8 += 8) {
            int4* dst = reinterpret_cast<int4*>(wrow + c8);
            dst[0] = make_int4((int)v[c8], (int)v[c8 + 1], (int)v[c8 + 2], (int)v[c8 + 3]);
            dst[1] = make_int4((int)v[c8 + 4], (int)v[c8 + 5], (int)v[c8 + 6], (int)v[c8 + 7]);
          }
        }
      } else if (TSTORE ? (t.m0 + sub * BM + 32 * q < p.M && n0 < p.N) : (m < p.M && n0 < p.N)) {
        // TSTORE: the condition is the same for the whole warp; rows and columns of the block
        // that lie past M or N are computed (from zero rows, clamped constants) and dropped by TMA
        uint8_t* obuf = sOut + (q + 4 * helper) * kOutBlock;
        if (TSTORE) {
          if (oc > 0) {  // this warp's previous store has read the buffer (the quarter's other warp works meanwhile)
            if (lane == 0) bulk_wait_read<0>();
            __syncwarp();
          }
        }
#pragma unroll
        for (int c8 = 0; c8 < 32; c8 += 8) {
          if (TSTORE || n0 + c8 < p.N) {  // N % 8 == 0: a group of 8 columns is all in or all out
            int acc[8];
            uint32_t o[4];
            const int4 cs0 = *reinterpret_cast<const int4*>(s_cs + c0 + c8);
            const int4 cs1 = *reinterpret_cast<const int4*>(s_cs + c0 + c8 + 4);
            const float4 sw0 = *reinterpret_cast<const float4*>(s_sw + c0 + c8);
            const float4 sw1 = *reinterpret_cast<const float4*>(s_sw + c0 + c8 + 4);
            const int cs[8] = {cs0.x, cs0.y, cs0.z, cs0.w, cs1.x, cs1.y, cs1.z, cs1.w};
            const float sw[8] = {sw0.x, sw0.y, sw0.z, sw0.w, sw1.x, sw1.y, sw1.z, sw1.w};
#pragma unroll
            for (int cc = 0; cc < 8; ++cc) acc[cc] = ((int)v[c8 + cc] - cs[cc]) >> 4;
#pragma unroll
            for (int cc = 0; cc < 8; cc += 2) {
              const float f0 = ((float)acc[cc] * sh) * sw[cc];
              const float f1 = ((float)acc[cc + 1] * sh) * sw[cc + 1];
              o[cc >> 1] = pack_bf16x2(f0, f1);
            }
            if (TSTORE) {
              // row `lane` of the block, 16-byte piece c8 / 8, in the 64-byte swizzle TMA expects
              *reinterpret_cast<uint4*>(obuf + lane * 64 + ((((c8 >> 3) ^ (lane >> 1)) & 3) << 4)) =
                  make_uint4(o[0], o[1], o[2], o[3]);
            } else {
              *reinterpret_cast<uint4*>(p.out + (size_t)m * p.N + n0 + c8) = make_uint4(o[0], o[1], o[2], o[3]);
            }
            if (p.acc_out != nullptr && (!TSTORE || (m < p.M && n0 + c8 < p.N))) {
              int4* dst = reinterpret_cast<int4*>(p.acc_out + (size_t)m * p.N + n0 + c8);
              dst[0] = make_int4(acc[0], acc[1], acc[2], acc[3]);
              dst[1] = make_int4(acc[4], acc[5], acc[6], acc[7]);
            }
          }
        }
        if (TSTORE) {
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) tma_store_2d(smem_u32(obuf), &map_b, n0, t.m0 + sub * BM + 32 * q);
          ++oc;
        }
      }
    }
    tc_fence_before();
    if (!released0) arrive_leader<PAIR>(bar_tempty);
    if (A8) arrive_leader<PAIR>(bar_tempty1);
    mbar_arrive(bar_edone);
    return true;
  };

  if (warp < kProdWarps) {
    // =============================================================== producers
    // Warp pw widens kRowsPerWarp rows of A (of the 256 of a stage) and as many rows of B;
    // lane -> (row % 8, packed 16-byte chunk): a quarter warp reads 128 contiguous packed bytes
    // and its two stores land on eight different 16-byte chunks of the swizzled rows.
    const int pw = warp;
    const int r7 = lane >> 2;
    const int c = lane & 3;
    const uint32_t sw_even = (uint32_t)(((2 * c) ^ r7) << 4);
    const uint32_t row0 = (uint32_t)(kRowsPerWarp * pw + r7) * 128u;          // widened: + i * 1024 for task i
    const uint32_t prow0 = (uint32_t)(kRowsPerWarp * pw + r7) * 64u + c * 16;  // packed:  + i * 512
    const uint32_t rowb0 = (uint32_t)(G::kRowsPerWarpB * pw + r7) * 128u;      // the same for this CTA's rows of B
    const uint32_t prowb0 = (uint32_t)(G::kRowsPerWarpB * pw + r7) * 64u + c * 16;
    // ---- processing side
    uint32_t it = 0;   // position in the ring of widened stages (dense and sparse steps)
    uint32_t pit = 0;  // position in the ring of packed stages (dense steps only)
    uint32_t pmul[kATasks], poff[kATasks];
#pragma unroll
    for (int i = 0; i < kATasks; ++i) {
      pmul[i] = 1;
      poff[i] = 0;
    }
    int pj = cl, pks = 0;  // work-list entry and K step being processed
    Tile pt = tile_of<PAIR, SPLITK>(p, pj, rank);
    // producer-side merge (PMERGE): lane l of the warp owns row 32 * pw + l of the stage and
    // keeps that row's 16 sparse values and positions of the coming K step in registers
    const int GKp = (p.K / p.b) * p.k;
    uint4 nrv = make_uint4(0, 0, 0, 0), nri = nrv;
    uint32_t pm_bank4[4] = {0, 0, 0, 0};
    if (PMERGE) {
#pragma unroll
      for (int w = 0; w < 4; ++w)
#pragma unroll
        for (int u = 0; u < 4; ++u) pm_bank4[w] |= (uint32_t)(((4 * w + u) >> p.log2k) * p.b) << (8 * u);
    }
    auto sparse_fetch = [&](const Tile& ft, int fks) {
      if (ft.m0 + 32 * pw + lane >= p.M) return;  // a row past M is not merged
      const int m = ft.m0 + 32 * pw + lane;
      const size_t o = (size_t)m * (size_t)GKp + (size_t)fks * 16;
      const uint8_t* ip = p.idx != nullptr ? p.idx + o : p.pos + (size_t)fks * 16;
      // (volatile: issued here, a whole K step before their use)
      asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                   : "=r"(nrv.x), "=r"(nrv.y), "=r"(nrv.z), "=r"(nrv.w)
                   : "l"(p.vals + o));
      asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                   : "=r"(nri.x), "=r"(nri.y), "=r"(nri.z), "=r"(nri.w)
                   : "l"(ip));
    };
    if (PMERGE && cl < nwork) sparse_fetch(pt, pt.k0);
    auto process = [&]() -> bool {
      // a single-sub-tile entry only has A rows 0..127; with pre-widened activations there is no A work at all
      const bool has_a = !A8 && (pt.nsub == 2 || pw < kProdWarps / 2);
      uint4 crv, cri;
      if (PMERGE) {
        crv = nrv;
        cri = nri;
        if (pks + 1 < KS) sparse_fetch(pt, pt.k0 + pks + 1);
        else if (pj + ncl < nwork) {
          const Tile nt = tile_of<PAIR, SPLITK>(p, pj + ncl, rank);
          sparse_fetch(nt, nt.k0);
        }
      }
      // ---- packed operands: wait for the TMA tiles, pull this thread's chunks into registers,
      //      hand the packed stage back
      const int ps = pit % NP;
      if (!WAIT_PF(bar_pfull + 8 * ps, (pit / NP) & 1u, abort_flag)) return false;
      uint4 ra[kATasks], rb[kBTasks];
      const uint8_t* pa = sPA + ps * kPackA + prow0;
      const uint8_t* pb = sPB + ps * kPackB + prowb0;
#pragma unroll
      for (int i = 0; i < kATasks; ++i) ra[i] = has_a ? *reinterpret_cast<const uint4*>(pa + i * 512) : make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int i = 0; i < kBTasks; ++i) rb[i] = *reinterpret_cast<const uint4*>(pb + i * 512);
      ++pit;

      const int s = it % NS;
      if (!WAIT_PE(bar_empty + 8 * s, ((it / NS) & 1u) ^ 1u, abort_flag)) return false;
      uint8_t* a_st = sA + s * kStageA;
      uint8_t* b_st = sB + s * kStageB;
      if (pks == 0 && has_a) {  // the rows' shifts change with the tile only
#pragma unroll
        for (int i = 0; i < kATasks; ++i) {
          const uint32_t e = p.shift[min(pt.m0 + kRowsPerWarp * pw + 8 * i + r7, p.M - 1)];
          pmul[i] = 1u << e;
          poff[i] = 0x01010101u * (128u - (8u << e));
        }
      }
      // ---- widen A: nibble -> u * 2^e + (128 - 8 * 2^e)
      if (has_a) {
#pragma unroll
        for (int i = 0; i < kATasks; ++i) {
          // eight rows that all lie past M (a launch of a few tokens: most of the tile) keep
          // whatever the stage holds: their products are never stored
          if (pt.m0 + kRowsPerWarp * pw + 8 * i >= p.M) continue;
          const uint32_t in[4] = {ra[i].x, ra[i].y, ra[i].z, ra[i].w};
          uint32_t ev[4], od[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t u = in[q] ^ 0x88888888u;
            ev[q] = (u & 0x0F0F0F0Fu) * pmul[i] + poff[i];
            od[q] = ((u >> 4) & 0x0F0F0F0Fu) * pmul[i] + poff[i];
          }
          uint8_t* dst = a_st + row0 + i * 1024;
          {
          *reinterpret_cast<uint4*>(dst + sw_even) = make_uint4(ev[0], ev[1], ev[2], ev[3]);
          *reinterpret_cast<uint4*>(dst + (sw_even ^ 16u)) = make_uint4(od[0], od[1], od[2], od[3]);
          }
        }
      }
      // ---- widen B: nibble -> 16 * code
#pragma unroll
      for (int i = 0; i < kBTasks; ++i) {
        const uint32_t in[4] = {rb[i].x, rb[i].y, rb[i].z, rb[i].w};
        uint32_t ev[4], od[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          ev[q] = (in[q] << 4) & 0xF0F0F0F0u;
          od[q] = in[q] & 0xF0F0F0F0u;
        }
        uint8_t* dst = b_st + rowb0 + i * 1024;
        {
        *reinterpret_cast<uint4*>(dst + sw_even) = make_uint4(ev[0], ev[1], ev[2], ev[3]);
        *reinterpret_cast<uint4*>(dst + (sw_even ^ 16u)) = make_uint4(od[0], od[1], od[2], od[3]);
        }
      }
      if (PMERGE && has_a) {
        __syncwarp();  // the warp's 32 rows are written: each lane now patches one of them
        const int row = 32 * pw + lane;
        if (pt.m0 + row < p.M) {
        const uint32_t swz = 0x01010101u * (uint32_t)((row & 7) << 4);
        uint8_t* rowp = a_st + row * 128;
        const uint32_t vw[4] = {crv.x, crv.y, crv.z, crv.w};
        const uint32_t iw[4] = {cri.x, cri.y, cri.z, cri.w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const uint32_t pos4 = (kpos4(iw[w]) + pm_bank4[w]) ^ swz;
          const uint32_t vx = vw[w] ^ 0x80808080u;
#pragma unroll
          for (int u = 0; u < 4; ++u) rowp[(pos4 >> (8 * u)) & 0xFFu] = (uint8_t)(vx >> (8 * u));
        }
        }
      }
      // The packed stage goes back to the TMA thread only now: shared-memory loads are
      // asynchronous, and an arrive issued right behind them could let the refill overtake
      // them; after the widening every loaded register has been consumed.
      mbar_arrive(bar_pempty + 8 * ps);
      fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor core's async reads
      if (STMA || PMERGE || A8) arrive_leader<PAIR>(bar_full + 8 * s);
      else mbar_arrive(bar_wfull + 8 * s);  // dynamic positions: the merge warps take over
      ++it;
      if (++pks == KS) {
        pks = 0;
        const int SS = STMA ? pt.ss : 0;  // sparse K steps of the work item just finished
        pj += ncl;
        if (pj < nwork) pt = tile_of<PAIR, SPLITK>(p, pj, rank);
        // The sparse K steps of the tile use the next SS ring slots (TMA fills them).  They are
        // waited for one by one, not skipped: a parity wait only tells the current phase from
        // the previous one, so no role may fall more than one use behind on any stage.
        for (int ss = 0; ss < SS; ++ss, ++it) {
          if (!mbar_wait(bar_empty + 8 * (it % NS), ((it / NS) & 1u) ^ 1u, abort_flag)) return false;
        }
      }
      return true;
    };

    // (Optional, see kProducersJoinEpilogue.)  After filling the first stages of a tile the ring
    // is full until the MMA thread moves on, and it moves on only when the previous tile's
    // accumulators have been read out: that is when the producers can lend a hand.
    const int my_tiles = (nwork - cl + ncl - 1) / ncl;
    const int join_step = (KS < NS ? KS : NS) - 1;
    bool ok = true;
    for (int ti = 0; ti < my_tiles && ok; ++ti) {
      for (int ks = 0; ks < KS && ok; ++ks) {
        ok = process();
        if (kProducersJoinEpilogue && ok && ks == join_step && ti > 0)
          ok = epilogue_share(tile_of<PAIR, SPLITK>(p, cl + (ti - 1) * ncl, rank), (uint32_t)(ti - 1), pw >> 2);
      }
    }
    if (kProducersJoinEpilogue && ok)
      epilogue_share(tile_of<PAIR, SPLITK>(p, cl + (my_tiles - 1) * ncl, rank), (uint32_t)(my_tiles - 1), pw >> 2);
  } else if (warp == kMmaWarp || warp == kMma2Warp) {
    // =============================================================== MMA issuer(s)
    // (the leader CTA's; the peer's MMA warp only holds its half of the tensor-memory allocation)
    // With TMA-delivered activations nothing but this loop paces the tensor pipe (~50 ns per
    // tcgen05.mma issue plus a barrier round trip and a commit per step against 560 ns of MMA
    // work), so two threads in two warps share it: each issues one sub-tile's MMAs and commits
    // for itself (the "empty" and "accumulators complete" barriers then expect two commits).
    const int sub_first = (A8 && warp == kMma2Warp) ? 1 : 0;
    if (lane == 0 && rank == 0 && (A8 || warp == kMmaWarp)) {
      constexpr uint32_t idesc = make_idesc(false, BM * PAIR);
      constexpr uint32_t idesc_sparse = make_idesc(true, BM * PAIR);
      uint32_t it = 0, tc = 0;
      uint32_t ph_dense = 0, ph_sparse = 0;  // per-stage phase bits of the two kinds of "full" barrier
      bool ok = true;
      for (int j = cl; j < nwork && ok; j += ncl, ++tc) {
        const Tile mt = tile_of<PAIR, SPLITK>(p, j, rank);
        const int nsub = mt.nsub;
        const int SS = STMA ? mt.ss : 0;
        // previous tile's accumulator(s) read out (both CTAs); with two issuing threads each waits for its own
        ok = wait_leader<PAIR>((A8 && warp == kMma2Warp) ? bar_tempty1 : bar_tempty, (tc & 1u) ^ 1u, abort_flag);
        if (!ok) break;
        tc_fence_after();
        // What a K step waits for: dense = the stage's "full" barrier (the producers or merge
        // warps; with TMA-delivered activations also both CTAs' tiles arrive there); sparse =
        // both CTAs' tile barriers.  With TMA-delivered activations the producers run well ahead
        // and this thread's own loop is what paces the tensor pipe, so it polls the NEXT step's
        // barrier once between the two sub-tiles' MMAs: the answer's latency hides behind the
        // issue of four MMAs.  (In the other modes the stage is usually not ready yet at that point and
        // the extra poll only delays the second sub-tile: measured 12 % slower.)
        bool seen = false;  // this step's barriers were already found complete
        for (int ks = 0; ks < KS + SS; ++ks, ++it) {
          const int s = it % NS;
          const bool sparse_step = ks >= KS;
          if (!seen) {
            if (!sparse_step) ok = wait_leader<PAIR>(bar_full + 8 * s, (ph_dense >> s) & 1u, abort_flag);
            if (ok && sparse_step) {
              ok = mbar_wait(bar_sfull + 8 * s, (ph_sparse >> s) & 1u, abort_flag);
              if (ok && PAIR == 2) ok = wait_leader<PAIR>(bar_sfullp + 8 * s, (ph_sparse >> s) & 1u, abort_flag);
            }
          }
          if (!ok) break;
          if (!sparse_step) ph_dense ^= 1u << s;
          if (sparse_step) ph_sparse ^= 1u << s;
          tc_fence_after();
          const uint64_t db = make_desc(smem_u32(sB + s * kStageB));
          const uint32_t id = sparse_step ? idesc_sparse : idesc;
          seen = false;
          const int sub_end = A8 ? (sub_first + 1 < nsub ? sub_first + 1 : nsub) : nsub;
          for (int sub = sub_first; sub < sub_end || (A8 && sub == sub_first); ++sub) {
            if (sub < nsub) {
              const uint64_t da = make_desc(smem_u32(sA + s * kStageA + sub * (BM * BK)));
#pragma unroll
              for (int kk = 0; kk < BK / 32; ++kk)  // 32 bytes of K per MMA: +2 in 16-byte address units
                umma_i8<PAIR>(tmem + ((INDEP && sparse_step) ? BN : sub * BN), da + 2 * kk, db + 2 * kk, id,
                              ((INDEP && sparse_step) ? (ks > KS || kk > 0) : (ks > 0 || kk > 0)) ? 1u : 0u);
            }
            if (A8 && sub == sub_first && ks + 1 < KS + SS) {
              const int s2 = (int)((it + 1) % NS);
              const bool sparse2 = ks + 1 >= KS;
              bool r = true;
              if (!sparse2) r = PAIR == 2 ? mbar_test_cluster(bar_full + 8 * s2, (ph_dense >> s2) & 1u)
                                          : mbar_test(bar_full + 8 * s2, (ph_dense >> s2) & 1u);
              if (r && sparse2) {
                r = mbar_test(bar_sfull + 8 * s2, (ph_sparse >> s2) & 1u);
                if (r && PAIR == 2) r = mbar_test_cluster(bar_sfullp + 8 * s2, (ph_sparse >> s2) & 1u);
              }
              seen = r;
            }
          }
          umma_commit<PAIR>(bar_empty + 8 * s);
        }
        if (ok) umma_commit<PAIR>(bar_tfull);
      }
    }
    __syncwarp();
  } else if (warp == kTmaWarp) {
    // =============================================================== TMA: packed dense tiles
    if (lane == 0) {
      uint32_t pit = 0;
      bool ok = true;
      for (int j = cl; j < nwork && ok; j += ncl) {
        const Tile t = tile_of<PAIR, SPLITK>(p, j, rank);
        for (int ks = 0; ks < KS && ok; ++ks, ++pit) {
          const int ps = pit % NP;
          ok = WAIT_T(bar_pempty + 8 * ps, ((pit / NP) & 1u) ^ 1u, abort_flag);
          if (!ok) break;
          // rows past M / N come back as zeros (code 0)
          mbar_expect_tx(bar_pfull + 8 * ps, (uint32_t)((A8 ? 0 : p.rows_a * (BK / 2)) + kPackB));
          if (!A8) tma_load_2d(smem_u32(sPA + ps * kPackA), &map_a4, (t.k0 + ks) * (BK / 2), t.m0, bar_pfull + 8 * ps);
          tma_load_2d(smem_u32(sPB + ps * kPackB), &map_b4, (t.k0 + ks) * (BK / 2), t.nb0, bar_pfull + 8 * ps);
        }
      }
    }
    __syncwarp();
  } else if (warp == kTmaSparseWarp) {
    // =============================================================== TMA: sparse K steps, or every
    // step's pre-widened activation tile
    if (ATMA && lane == 0) {
      uint32_t it = 0;
      // The leader's MMA thread cannot watch the peer's barriers, so the peer's thread tells it
      // when each of its tiles has landed.  It does so while waiting for the next free slot
      // (never blocking on a load it has just issued), oldest load first.
      const bool forwards = PAIR == 2 && rank != 0;
      uint32_t fq[NS];            // slots of the loads not yet reported, in issue order
      uint32_t fq_head = 0, fq_n = 0, ph_fwd = 0;
      auto try_forward = [&]() {
        while (fq_n > 0) {
          const uint32_t fs = fq[fq_head % NS];
          if (!mbar_test(bar_sfull + 8 * fs, (ph_fwd >> fs) & 1u)) break;
          ph_fwd ^= 1u << fs;
          mbar_arrive_cta((A8 ? bar_full : bar_sfullp) + 8 * fs, 0);
          ++fq_head;
          --fq_n;
        }
      };
      bool ok = true;
      for (int j = cl; j < nwork && ok; j += ncl) {
        const Tile t = tile_of<PAIR, SPLITK>(p, j, rank);
        const int SS = STMA ? t.ss : 0;
        // every ring slot is waited for in order (see the producers); only the sparse ones are filled
        for (int step = 0; step < KS + SS && ok; ++step, ++it) {
          const int s = it % NS;
          const uint32_t par = ((it / NS) & 1u) ^ 1u;
          if (!forwards) {
            ok = WAIT_T(bar_empty + 8 * s, par, abort_flag);
          } else {
            ok = false;
            for (uint32_t n = 0; n < kSpinLimit; ++n) {
              if (mbar_test(bar_empty + 8 * s, par)) {
                ok = true;
                break;
              }
              try_forward();
              if ((n & 1023u) == 1023u && *abort_flag) break;
            }
            if (!ok) *abort_flag = 1;
          }
          if (!ok) continue;
          if (A8) {
            // the merged 8-bit activations of this K step (rows past M come back as zeros).  The
            // leader's tile completes on the stage's "full" barrier itself, the peer's on its own
            // barrier, from where it is reported to that same "full": the MMA thread then has a
            // single barrier to look at per step.
            const uint32_t abar = (forwards ? bar_sfull : bar_full) + 8 * s;
            mbar_expect_tx(abar, (uint32_t)kStageA);
            tma_load_2d(smem_u32(sA + s * kStageA), &map_a, (t.k0 + step) * BK, t.m0, abar);
          } else {
            if (step < KS) continue;
            const int ss = step - KS;
            // rows past M / N and columns past G*k are filled with zeros by the TMA unit
            mbar_expect_tx(bar_sfull + 8 * s, (uint32_t)(p.rows_a * BK + kStageB));
            tma_load_2d(smem_u32(sA + s * kStageA), &map_a, ss * BK, t.m0, bar_sfull + 8 * s);
            tma_load_2d(smem_u32(sB + s * kStageB), &map_b, ss * BK, t.nb0, bar_sfull + 8 * s);
          }
          if (forwards) {
            fq[(fq_head + fq_n) % NS] = (uint32_t)s;
            ++fq_n;
            try_forward();
          }
        }
      }
      // report what is still in flight
      for (uint32_t n = 0; forwards && ok && fq_n > 0 && n < kSpinLimit; ++n) {
        try_forward();
        if ((n & 1023u) == 1023u && *abort_flag) break;
      }
    }
    __syncwarp();
  } else {
    // =============================================================== epilogue
    // 0..127 among the epilogue threads (128..255: the four extra warps of the 8-bit activation mode)
    const int et = warp > kMma2Warp ? 128 + tid - (kMma2Warp + 1) * 32 : tid - (kMmaWarp + 1) * 32;
    // merge state (dynamic positions): word tasks tt = et + 128*jj -> (row tt / words-per-row, word)
    const int m_GK = (p.K / p.b) * p.k;
    const int m_nb = (BK / p.b) * p.k;  // sparse entries per row per K step
    const bool m_word_path = !STMA && !PMERGE && !A8 && p.log2k >= 0;
    const int m_nw_log = m_word_path ? (31 - __clz(m_nb >> 2)) : 0;
    const int m_ntask = m_word_path ? (2 * BM << m_nw_log) / 128 : 0;  // per thread for a 256-row stage
    const bool m_prefetch = m_ntask <= kMergeTasks;
    uint32_t m_bank4[kMergeTasks], mv[kMergeTasks], mi[kMergeTasks];
#pragma unroll
    for (int jj = 0; jj < kMergeTasks; ++jj) {
      const int q = (et + 128 * jj) & ((1 << m_nw_log) - 1);
      uint32_t b4 = 0;
      if (m_word_path) {
#pragma unroll
        for (int u = 0; u < 4; ++u) b4 |= (uint32_t)(((4 * q + u) >> p.log2k) * p.b) << (8 * u);
      }
      m_bank4[jj] = b4;
      mv[jj] = mi[jj] = 0;
    }
    if (m_word_path && m_prefetch) {  // sparse words of the very first step
      const Tile t0 = tile_of<PAIR, SPLITK>(p, cl, rank);
#pragma unroll
      for (int jj = 0; jj < kMergeTasks; ++jj) {
        const int tt = et + 128 * jj;
        if (jj < m_ntask && (tt >> m_nw_log) < t0.nsub * BM) {
          const int m = min(t0.m0 + (tt >> m_nw_log), p.M - 1);
          const uint32_t o = (uint32_t)m * (uint32_t)m_GK + (uint32_t)t0.k0 * (uint32_t)m_nb + 4 * (tt & ((1 << m_nw_log) - 1));
          mv[jj] = __ldg(reinterpret_cast<const uint32_t*>(p.vals + o));
          mi[jj] = p.idx != nullptr ? __ldg(reinterpret_cast<const uint32_t*>(p.idx + o))
                                    : __ldg(reinterpret_cast<const uint32_t*>(p.pos + t0.k0 * m_nb + 4 * (tt & ((1 << m_nw_log) - 1))));
        }
      }
    }
    uint32_t mit = 0;  // position in the ring of widened stages
    uint32_t tc = 0;
    for (int j = cl; j < nwork; j += ncl, ++tc) {
      const Tile t = tile_of<PAIR, SPLITK>(p, j, rank);
      // the tile's column constants are fetched while the main loop is still running
      for (int cc = et; cc < BN; cc += (A8 ? kEpiWarpsA8 : kEpiWarps) * 32) {
        const int n = min(t.n0 + cc, p.N - 1);
        s_cs[cc] = 2048 * __ldg(p.colsum + n);
        s_sw[cc] = __ldg(p.s_w + n);
      }
      if (!STMA && !PMERGE && !A8) {
        // ---- dynamic positions (or static ones TMA cannot fetch): these warps, idle until the
        //      tile's accumulators are complete, merge the sparse INT8 entries into every widened
        //      A stage and only then hand it to the MMA thread
        bool ok = true;
        for (int ks = 0; ks < KS && ok; ++ks, ++mit) {
          const int s = mit % NS;
          // sparse words of this step (prefetched) ...
          uint32_t cv[kMergeTasks], ci[kMergeTasks];
          if (m_word_path && m_prefetch) {
#pragma unroll
            for (int jj = 0; jj < kMergeTasks; ++jj) {
              cv[jj] = mv[jj];
              ci[jj] = mi[jj];
            }
            // ... and the next step's (next tile's first step at the end of this one)
            int nj = j, nks = ks + 1;
            if (nks == KS) {
              nks = 0;
              nj += ncl;
            }
            if (nj < nwork) {
              const Tile nt = nks == 0 ? tile_of<PAIR, SPLITK>(p, nj, rank) : t;
#pragma unroll
              for (int jj = 0; jj < kMergeTasks; ++jj) {
                const int tt = et + 128 * jj;
                if (jj < m_ntask && (tt >> m_nw_log) < nt.nsub * BM) {
                  const int m = min(nt.m0 + (tt >> m_nw_log), p.M - 1);
                  const uint32_t o = (uint32_t)m * (uint32_t)m_GK + (uint32_t)(nt.k0 + nks) * (uint32_t)m_nb + 4 * (tt & ((1 << m_nw_log) - 1));
                  mv[jj] = __ldg(reinterpret_cast<const uint32_t*>(p.vals + o));
                  mi[jj] = p.idx != nullptr
                               ? __ldg(reinterpret_cast<const uint32_t*>(p.idx + o))
                               : __ldg(reinterpret_cast<const uint32_t*>(p.pos + (nt.k0 + nks) * m_nb + 4 * (tt & ((1 << m_nw_log) - 1))));
                }
              }
            }
          }
          ok = mbar_wait(bar_wfull + 8 * s, (mit / NS) & 1u, abort_flag);
          if (!ok) break;
          uint8_t* a_st = sA + s * kStageA;
          if (m_word_path && m_prefetch) {
#pragma unroll
            for (int jj = 0; jj < kMergeTasks; ++jj) {
              const int tt = et + 128 * jj;
              const int row = tt >> m_nw_log;
              if (jj < m_ntask && row < t.nsub * BM) {
                const uint32_t pos4 = (kpos4(ci[jj]) + m_bank4[jj]) ^ (0x01010101u * (uint32_t)((row & 7) << 4));
                const uint32_t vx = cv[jj] ^ 0x80808080u;
                uint8_t* rowp = a_st + row * 128;
#pragma unroll
                for (int u = 0; u < 4; ++u) rowp[(pos4 >> (8 * u)) & 0xFFu] = (uint8_t)(vx >> (8 * u));
              }
            }
          } else if (m_word_path) {  // many entries per step: word loads without register prefetch
            for (int tt = et; tt < ((t.nsub * BM) << m_nw_log); tt += 128) {
              const int row = tt >> m_nw_log, q = tt & ((1 << m_nw_log) - 1);
              const int m = min(t.m0 + row, p.M - 1);
              const uint32_t o = (uint32_t)m * (uint32_t)m_GK + (uint32_t)(t.k0 + ks) * (uint32_t)m_nb + 4 * q;
              const uint32_t vw = __ldg(reinterpret_cast<const uint32_t*>(p.vals + o));
              const uint32_t iw = p.idx != nullptr ? __ldg(reinterpret_cast<const uint32_t*>(p.idx + o))
                                                   : __ldg(reinterpret_cast<const uint32_t*>(p.pos + (t.k0 + ks) * m_nb + 4 * q));
              uint32_t b4 = 0;
#pragma unroll
              for (int u = 0; u < 4; ++u) b4 |= (uint32_t)(((4 * q + u) >> p.log2k) * p.b) << (8 * u);
              const uint32_t pos4 = (kpos4(iw) + b4) ^ (0x01010101u * (uint32_t)((row & 7) << 4));
              const uint32_t vx = vw ^ 0x80808080u;
              uint8_t* rowp = a_st + row * 128;
#pragma unroll
              for (int u = 0; u < 4; ++u) rowp[(pos4 >> (8 * u)) & 0xFFu] = (uint8_t)(vx >> (8 * u));
            }
          } else {  // any k: byte-wise
            for (int tt = et; tt < t.nsub * BM * m_nb; tt += 128) {
              const int row = tt / m_nb, i = tt - row * m_nb;
              const int m = min(t.m0 + row, p.M - 1);
              const int bank = i / p.k, slot_i = i - bank * p.k;
              const int g = (t.k0 + ks) * (BK / p.b) + bank;
              const size_t entry = (size_t)m * m_GK + (size_t)g * p.k + slot_i;
              const uint32_t local = p.idx != nullptr ? p.idx[entry] : p.pos[(size_t)g * p.k + slot_i];
              const uint32_t kp = (kpos1(local) + (uint32_t)(bank * p.b)) ^ (uint32_t)((row & 7) << 4);
              a_st[row * 128 + kp] = (uint8_t)((uint8_t)p.vals[entry] ^ 0x80u);
            }
          }
          fence_proxy_async_smem();
          arrive_leader<PAIR>(bar_full + 8 * s);
        }
        if (!ok) break;
      }
      if (!epilogue_share(t, tc, A8 ? (warp > kMma2Warp ? 1 : 0) : (kProducersJoinEpilogue ? 2 : 0))) break;
      // the constants may be replaced only when every helper is done with them
      if (!mbar_wait(bar_edone, tc & 1u, abort_flag)) break;
    }
    if (TSTORE && lane == 0) bulk_wait_all();  // the staged blocks have left before the CTA does
  }

  tc_fence_before();
  __syncthreads();
  // Neither CTA of a pair may leave (or free tensor memory) while the other can still arrive on
  // its barriers or have MMAs reading its shared memory.
  if (PAIR == 2) cluster_sync_all();
  if (SPLITK && PAIR == 1 && p.ws == nullptr) {
    // Clustered split-K: the cluster's CTAs hold the parts of one column tile.  Every thread of
    // every CTA gets here, whatever happened before (an aborted wait only leaves garbage to
    // add), so the two cluster barriers cannot be missed by anyone.  CTA r of the cluster then
    // adds all parts of its share of the columns, read from the peers' shared memory, and runs
    // the same epilogue arithmetic as the one-kernel path (integer sums: order-free).
    cluster_sync_all();
    const int parts = p.splits, r = (int)cluster_ctarank();
    const int n_tile = ((int)blockIdx.x / parts) * BN;
    const int m_base = (p.mu - 1) * BM;               // the (only) row unit of a few-row launch
    const int groups_per_row = (BN / 8) / parts;      // groups of eight columns in this CTA's share
    const int rows = p.M - m_base;
    for (int g = tid; g < rows * groups_per_row; g += (int)blockDim.x) {
      const int row = g / groups_per_row, g8 = r * groups_per_row + g % groups_per_row;
      const int m = m_base + row, n = n_tile + 8 * g8;
      if (n >= p.N) continue;
      int v[8] = {0, 0, 0, 0, 0, 0, 0, 0};
      const uint32_t base = smem_u32(smem) + (uint32_t)row * (BN * 4);
      for (int sp = 0; sp < parts; ++sp) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint32_t laddr = base + (uint32_t)(((2 * g8 + h) ^ (row & 7)) << 4);
          int4 a;
          asm volatile(
              "{\n\t.reg .b32 ra;\n\t"
              "mapa.shared::cluster.u32 ra, %4, %5;\n\t"
              "ld.shared::cluster.v4.s32 {%0, %1, %2, %3}, [ra];\n\t}"
              : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w)
              : "r"(laddr), "r"(sp)
              : "memory");
          v[4 * h] += a.x; v[4 * h + 1] += a.y; v[4 * h + 2] += a.z; v[4 * h + 3] += a.w;
        }
      }
      const float sh = p.s_hi[m];
      int acc[8];
      uint32_t o[4];
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[c] = (v[c] - 2048 * p.colsum[n + c]) >> 4;
#pragma unroll
      for (int c = 0; c < 8; c += 2)
        o[c >> 1] = pack_bf16x2(((float)acc[c] * sh) * p.s_w[n + c], ((float)acc[c + 1] * sh) * p.s_w[n + c + 1]);
      *reinterpret_cast<uint4*>(p.out + (size_t)m * p.N + n) = make_uint4(o[0], o[1], o[2], o[3]);
      if (p.acc_out != nullptr) {
        int4* dst = reinterpret_cast<int4*>(p.acc_out + (size_t)m * p.N + n);
        dst[0] = make_int4(acc[0], acc[1], acc[2], acc[3]);
        dst[1] = make_int4(acc[4], acc[5], acc[6], acc[7]);
      }
    }
    cluster_sync_all();  // nobody leaves while a peer may still read its partial sums
  }
  if (tid == 0 && *abort_flag) atomicExch(p.status, (int)SQ_ERR_TIMEOUT);
  if (warp == kMmaWarp) tmem_dealloc<PAIR>(tmem, 2 * BN);
#undef rank
#undef cl
#undef ncl
}

// Merged 8-bit activations for kModeA8: a8[m][j'] = the operand byte the producers would put into
// the widened A stage (dense: offset-binary nibble * 2^e + bias; sparse: vals ^ 0x80), j' = the
// position of element j in the MMA's K order ([16 even | 16 odd] per 32 elements).  One thread
// per 32-element block: 16 packed bytes in, 32 operand bytes out, then the sparse entries of its
// bank that fall into the block are patched in.
__global__ void __launch_bounds__(256) expand_a8_kernel(const uint8_t* __restrict__ dq4, const int8_t* __restrict__ vals,
                                                        const uint8_t* __restrict__ idx,
                                                        const uint8_t* __restrict__ pos,
                                                        const uint8_t* __restrict__ shift, int64_t M, int K, int b,
                                                        int k, uint8_t* __restrict__ a8) {
  __shared__ __align__(16) uint8_t stage[256 * 32];
  const int blocks_per_row = K / 32;
  const int64_t total = M * blocks_per_row;
  const int GK = (K / b) * k;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t m = t / blocks_per_row;
    const int blk = (int)(t % blocks_per_row);  // elements 32*blk .. 32*blk+31 of the row
    const uint32_t e = shift[m];
    const uint32_t pmul = 1u << e, poff = 0x01010101u * (128u - (8u << e));
    const uint4 in = *reinterpret_cast<const uint4*>(dq4 + m * (K / 2) + blk * 16);
    const uint32_t w[4] = {in.x, in.y, in.z, in.w};
    uint32_t o[8];  // bytes 0..15: even elements, 16..31: odd elements
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint32_t u = w[q] ^ 0x88888888u;
      o[q] = (u & 0x0F0F0F0Fu) * pmul + poff;
      o[4 + q] = ((u >> 4) & 0x0F0F0F0Fu) * pmul + poff;
    }
    // the 32 operand bytes go through shared memory, where the sparse entries of the bank this
    // block lies in are patched in with byte stores, and leave as two 16-byte stores
    uint8_t* orow = stage + threadIdx.x * 32;
    uint4* sdst = reinterpret_cast<uint4*>(orow);
    sdst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    sdst[1] = make_uint4(o[4], o[5], o[6], o[7]);
    const int g = (blk * 32) / b, off = (blk * 32) % b;  // bank, and the block's first element inside it
    const int8_t* v = vals + m * GK + g * k;
    const uint8_t* ix = idx != nullptr ? idx + m * GK + g * k : pos + g * k;
    if ((k & 7) == 0 && ((reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(ix)) & 7) == 0) {
      for (int i8 = 0; i8 < k; i8 += 8) {  // eight entries per pair of 8-byte loads
        const uint2 iw = *reinterpret_cast<const uint2*>(ix + i8);
        const uint2 vw = *reinterpret_cast<const uint2*>(v + i8);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int jj = (int)(((i < 4 ? iw.x : iw.y) >> (8 * (i & 3))) & 0xFFu) - off;
          const uint32_t byte = (((i < 4 ? vw.x : vw.y) >> (8 * (i & 3))) & 0xFFu) ^ 0x80u;
          if (jj >= 0 && jj < 32) orow[((jj & 1) << 4) | (jj >> 1)] = (uint8_t)byte;
        }
      }
    } else {
      for (int i = 0; i < k; ++i) {
        const int jj = (int)ix[i] - off;
        if (jj >= 0 && jj < 32) orow[((jj & 1) << 4) | (jj >> 1)] = (uint8_t)((uint8_t)v[i] ^ 0x80u);
      }
    }
    uint4* dst = reinterpret_cast<uint4*>(a8 + m * K + blk * 32);
    dst[0] = sdst[0];
    dst[1] = sdst[1];
  }
}

// Split-K, second kernel: out[m, n] from the `splits` raw partial sums of every accumulator
// (the same integer and fp32 operations, in the same order, as the one-kernel epilogue).
__global__ void __launch_bounds__(256) splitk_finish_kernel(const int32_t* __restrict__ ws, int splits, int M, int N,
                                                            const int32_t* __restrict__ colsum,
                                                            const float* __restrict__ s_hi,
                                                            const float* __restrict__ s_w, uint16_t* __restrict__ out,
                                                            int32_t* __restrict__ acc_out) {
  const int64_t groups = (int64_t)M * (N / 8);
  for (int64_t gidx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; gidx < groups;
       gidx += (int64_t)gridDim.x * blockDim.x) {
    const int m = (int)(gidx / (N / 8)), n = (int)(gidx % (N / 8)) * 8;
    int v[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int sp = 0; sp < splits; ++sp) {
      const int4* src = reinterpret_cast<const int4*>(ws + ((size_t)sp * M + m) * N + n);
      const int4 a = src[0], b = src[1];
      v[0] += a.x; v[1] += a.y; v[2] += a.z; v[3] += a.w;
      v[4] += b.x; v[5] += b.y; v[6] += b.z; v[7] += b.w;
    }
    const float sh = s_hi[m];
    int acc[8];
    uint32_t o[4];
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] = (v[c] - 2048 * colsum[n + c]) >> 4;
#pragma unroll
    for (int c = 0; c < 8; c += 2)
      o[c >> 1] = pack_bf16x2(((float)acc[c] * sh) * s_w[n + c], ((float)acc[c + 1] * sh) * s_w[n + c + 1]);
    *reinterpret_cast<uint4*>(out + (size_t)m * N + n) = make_uint4(o[0], o[1], o[2], o[3]);
    if (acc_out != nullptr) {
      int4* dst = reinterpret_cast<int4*>(acc_out + (size_t)m * N + n);
      dst[0] = make_int4(acc[0], acc[1], acc[2], acc[3]);
      dst[1] = make_int4(acc[4], acc[5], acc[6], acc[7]);
    }
  }
}

// Split-K (at most 128 rows): how many parts of K per output tile, given the workspace.  With
// few rows a launch has only N/256 tiles and each walks all of K at about a microsecond per
// step (cold weight rows), so K is cut into up to 8 parts that run on other SMs at the same time.
static int choose_splits(int64_t M, int64_t N, int64_t K, int sms, size_t ws_bytes) {
  if (M > BM) return 1;
  const int64_t tiles_n = (N + BN - 1) / BN, ks = K / BK;
  for (int sp = 8; sp >= 2; sp /= 2) {
    if (tiles_n * sp <= sms && ks % sp == 0 && ks / sp >= 2 && (size_t)sp * M * N * 4 <= ws_bytes) return sp;
  }
  return 1;
}

// More than 128 rows: with M*K bytes of workspace the activations are expanded once into merged
// 8-bit operands (kModeA8) instead of being widened, and merged, again for every column tile.
// Worth the extra pass from a few column tiles on, for dynamic positions (it replaces the merge:
// 2640 against 1760 TOPS at M = 4096, N = K = 8192) and for static ones (it replaces the sparse K
// steps and two thirds of the widening: 2580 against 2480).
static bool use_a8(bool /*is_static*/, int64_t M, int64_t N, int64_t K, size_t ws_bytes) {
  return M > BM && (N + BN - 1) / BN >= 4 && (size_t)M * (size_t)K <= ws_bytes;
}

size_t gemm_workspace_bytes(int b, int k, bool is_static, bool indep, int64_t M, int64_t N, int64_t K) {
  if (indep) return 0;  // two accumulators: neither a merged 8-bit operand nor split-K is built for it
  if (gemm_stream_serves(b, k, is_static, M, N, K)) return 0;  // the weight-streaming kernel needs none
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  if (M > BM) return use_a8(is_static, M, N, K, ~(size_t)0) ? (size_t)M * K : 0;
  const int sp = choose_splits(M, N, K, sms, ~(size_t)0);
  return sp > 1 ? (size_t)sp * M * N * 4 : 0;
}

cudaError_t launch_expand_a8(int b, int k, const sq_encoded& A, const uint8_t* positions, int64_t M, int64_t K,
                             uint8_t* a8, cudaStream_t st) {
  int dev = 0, sms = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;
  const int64_t units = M * (K / 32);
  int64_t blocks = (units + 255) / 256;
  if (blocks > 32 * (int64_t)sms) blocks = 32 * (int64_t)sms;
  expand_a8_kernel<<<(unsigned)blocks, 256, 0, st>>>(A.dq4, A.vals, positions == nullptr ? A.idx : nullptr, positions,
                                                    A.shift, M, (int)K, b, k, a8);
  return cudaGetLastError();
}

cudaError_t launch_gemm(int b, int k, bool indep, const sq_encoded& A, const sq_weights& W,
                        const uint8_t* positions, int64_t M, int64_t N, int64_t K, uint16_t* out,
                        int32_t* acc_out, int* status, void* workspace, size_t workspace_bytes, bool allow_stream,
                        cudaStream_t st, bool a8_ready) {
  // (the few-token kernel fetches static positions through TMA: 16-byte aligned ones only)
  if (allow_stream && !indep && (reinterpret_cast<uintptr_t>(positions) & 15) == 0 && gemm_stream_serves(b, k, positions != nullptr, M, N, K))
    return launch_gemm_stream(b, k, A, W, positions, M, N, K, out, acc_out, status, st);
  GemmParams p;
  p.dq4 = A.dq4;
  p.vals = A.vals;
  p.idx = positions == nullptr ? A.idx : nullptr;
  p.pos = positions;
  p.s_hi = A.s_hi;
  p.s_lo = A.s_lo;
  p.shift = A.shift;
  p.wq4 = W.wq4;
  p.s_w = W.s_w;
  p.colsum = W.colsum;
  p.out = out;
  p.acc_out = acc_out;
  p.status = status;
  p.M = (int)M;
  p.N = (int)N;
  p.K = (int)K;
  p.b = b;
  p.k = k;
  // the kernel addresses the packed tensors with 32-bit byte offsets
  const int64_t GK = (K / b) * k;
  if (M * (K / 2) >= (1ll << 32) || N * (K / 2) >= (1ll << 32) || M * GK >= (1ll << 32)) return cudaErrorInvalidValue;
  // 32-bit word loads of the sparse entries need k a power of two, at least four entries per
  // row per K step and 4-byte aligned row starts; anything else takes the byte-wise path.
  const int nb = (BK / b) * k;
  const bool pow2 = (k & (k - 1)) == 0;
  p.log2k = -1;
  if (pow2 && nb >= 4 && GK % 4 == 0) {
    int l = 0;
    while ((1 << l) < k) ++l;
    p.log2k = l;
  }

  static std::atomic<int> sm_count_of[64];
  static std::atomic<int> pair_slots[64][5];  // CTA pairs that can be resident at once, per kernel variant
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  int sms = sm_count_of[dev].load(std::memory_order_acquire);
  if (sms == 0) {
    err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (err != cudaSuccess) return err;
    sm_count_of[dev].store(sms, std::memory_order_release);
  }
  const bool stma = positions != nullptr && GK % 16 == 0;
  // 16 sparse entries per row and K step, fetched with aligned 16-byte loads: the producers merge
  const uint8_t* pos_src = positions == nullptr ? A.idx : positions;
  const bool pmerge = !stma && nb == 16 && p.log2k >= 0 && GK % 16 == 0 &&
                      ((reinterpret_cast<uintptr_t>(A.vals) | reinterpret_cast<uintptr_t>(pos_src)) & 15) == 0;
  if (indep && !stma) return cudaErrorNotSupported;
  if (indep) workspace = nullptr;
  const bool a8 = workspace != nullptr && use_a8(positions != nullptr, M, N, K, workspace_bytes);
  if (a8_ready && !a8) {  // the caller's merged operand is of no use to this shape: leave it untouched
    workspace = nullptr;
    workspace_bytes = 0;
  }
  const int mode = indep ? kModeIndep : a8 ? kModeA8 : (stma ? kModeTma : (pmerge ? kModeMergeProd : kModeMergeEpi));
  // One CTA per tile for at most 128 rows (a second CTA would have no rows); CTA pairs otherwise.
  const int pair = M > BM ? 2 : 1;
  int slots = sms;  // tiles in flight at once
  if (pair == 2) {
    if (pair_slots[dev][mode].load(std::memory_order_acquire) == 0) {
      std::lock_guard<std::mutex> lock(setup_mutex());
      cudaLaunchConfig_t qc;
      memset(&qc, 0, sizeof(qc));
      cudaLaunchAttribute qa[1];
      qa[0].id = cudaLaunchAttributeClusterDimension;
      qa[0].val.clusterDim.x = 2;
      qa[0].val.clusterDim.y = 1;
      qa[0].val.clusterDim.z = 1;
      qc.gridDim = dim3((unsigned)(sms & ~1), 1, 1);
      qc.blockDim = dim3(threads_of(mode), 1, 1);
      qc.dynamicSmemBytes = (mode == kModeA8 ? Geo<2, kModeA8>::kSmemBytes : Geo<2>::kSmemBytes);
      qc.attrs = qa;
      qc.numAttrs = 1;
      int n = 0;
      const void* fn = mode == kModeIndep ? (const void*)gemm_kernel<2, kModeIndep, false>
                       : mode == kModeTma ? (const void*)gemm_kernel<2, kModeTma, false>
                       : mode == kModeMergeProd ? (const void*)gemm_kernel<2, kModeMergeProd, false>
                       : mode == kModeA8 ? (const void*)gemm_kernel<2, kModeA8, false>
                                         : (const void*)gemm_kernel<2, kModeMergeEpi, false>;
      err = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (mode == kModeA8 ? Geo<2, kModeA8>::kSmemBytes : Geo<2>::kSmemBytes));
      if (err == cudaSuccess) err = cudaOccupancyMaxActiveClusters(&n, fn, &qc);
      if (err != cudaSuccess) return err;
      if (n < 1) return cudaErrorLaunchOutOfResources;
      pair_slots[dev][mode].store(n, std::memory_order_release);
    }
    slots = pair_slots[dev][mode].load(std::memory_order_acquire);
  }

  // Work list: tiles of two row units per CTA while they fill whole waves of the slots; the
  // remainder of the row pairs is cut into tiles of one row unit so the last wave spreads over
  // twice as many slots.  (Row unit: 128 rows per CTA of the tile.)
  const int U = BM * pair;
  p.rows_a = pair == 1 ? (int)((M + 7) / 8 * 8) : 2 * BM;
  p.mu = (int)((M + U - 1) / U);
  p.mp = p.mu / 2;
  p.tiles_n = (int)((N + BN - 1) / BN);
  const int64_t pair_tiles = (int64_t)p.mp * p.tiles_n;
  int64_t as_pairs = (pair_tiles / slots) * slots;
  {
    // Cutting the remainder pays only if it saves waves: a one-sub-tile tile costs about 0.65
    // of a two-sub-tile one (it widens the same weight stage for half the MMA work).
    const int64_t rem = pair_tiles - as_pairs;
    const double cost_whole = (double)((rem + slots - 1) / slots);
    const double cost_cut = 0.65 * (double)((2 * rem + slots - 1) / slots);
    if (cost_whole <= cost_cut) as_pairs = pair_tiles;
  }
  if (indep) as_pairs = 0;  // the second accumulator takes the second sub-tile's tensor-memory columns
  p.n_pairs = (int)as_pairs;
  p.n_split = (int)(2 * (pair_tiles - as_pairs));
  // split-K (one CTA per tile, at most 128 rows, caller-provided workspace)
  p.splits = 1;
  p.ws = nullptr;
  p.KS = (int)(K / BK);
  int cluster_x = pair;  // CTAs per thread-block cluster
  if (pair == 1 && workspace != nullptr) {
    const int sp = choose_splits(M, N, K, sms, workspace_bytes);
    if (sp > 1) {
      p.splits = sp;
      p.ws = static_cast<int32_t*>(workspace);
      p.KS = (int)(K / BK / sp);
    }
  }
  if (pair == 1 && !indep && p.ws == nullptr) {  // also: a workspace too small for two parts
    // No workspace: the parts of a column tile run as one thread-block cluster and add their
    // partial sums through distributed shared memory at the end of the kernel (no second kernel).
    // The largest cluster size whose clusters can ALL be resident at once (a cluster needs its
    // SMs inside one GPC, so fewer clusters of 8 fit than SMs / 8; a second wave would cost more
    // than the longer K walk of a smaller cluster).
    static std::atomic<int> resident[64][3][4];  // per device, kernel variant, log2(cluster size): 0 = not asked yet
    const int variant = mode == kModeTma ? 0 : (mode == kModeMergeProd ? 1 : 2);
    const int64_t tiles_n = (N + BN - 1) / BN, ks = K / BK;
    for (int sp = 8, lg = 3; sp >= 2; sp /= 2, --lg) {
      if (tiles_n * sp > sms || ks % sp != 0 || ks / sp < 2) continue;
      if (resident[dev][variant][lg].load(std::memory_order_acquire) == 0) {
        std::lock_guard<std::mutex> lock(setup_mutex());
        cudaLaunchConfig_t qc;
        memset(&qc, 0, sizeof(qc));
        cudaLaunchAttribute qa[1];
        qa[0].id = cudaLaunchAttributeClusterDimension;
        qa[0].val.clusterDim.x = (unsigned)sp;
        qa[0].val.clusterDim.y = 1;
        qa[0].val.clusterDim.z = 1;
        qc.gridDim = dim3((unsigned)(sms / sp * sp), 1, 1);
        qc.blockDim = dim3(kThreads, 1, 1);
        qc.dynamicSmemBytes = Geo<1>::kSmemBytes;
        qc.attrs = qa;
        qc.numAttrs = 1;
        const void* fn = variant == 0 ? (const void*)gemm_kernel<1, kModeTma, true>
                         : variant == 1 ? (const void*)gemm_kernel<1, kModeMergeProd, true>
                                        : (const void*)gemm_kernel<1, kModeMergeEpi, true>;
        int n = 0;
        err = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<1>::kSmemBytes);
        if (err == cudaSuccess) err = cudaOccupancyMaxActiveClusters(&n, fn, &qc);
        if (err != cudaSuccess) return err;
        resident[dev][variant][lg].store(n > 0 ? n : -1, std::memory_order_release);
      }
      if (resident[dev][variant][lg].load(std::memory_order_acquire) >= tiles_n) {
        p.splits = sp;
        p.KS = (int)(ks / sp);
        cluster_x = sp;
        break;
      }
    }
  }
  p.n_singles = p.n_split + (p.mu & 1) * p.tiles_n * p.splits;
  const int64_t nwork = (int64_t)p.n_pairs + p.n_singles;
  const unsigned grid = (unsigned)(nwork < slots ? nwork : slots) * (unsigned)pair;

  // Static positions: the sparse product runs as extra K steps over vals [M, G*k] and
  // w_sparse [N, G*k], fetched by TMA.  A TMA row pitch must be a multiple of 16 bytes; any
  // other G*k falls back to merging the entries into the dense tile like dynamic positions.
  CUtensorMap map_a, map_b, map_a4, map_b4;
  memset(&map_a, 0, sizeof(map_a));
  memset(&map_b, 0, sizeof(map_b));
  static std::atomic<PFN_cuTensorMapEncodeTiled> encode_fn{nullptr};
  PFN_cuTensorMapEncodeTiled encode = encode_fn.load(std::memory_order_acquire);
  if (encode == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    err = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (err != cudaSuccess) return err;
    if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
    encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(fn);
    encode_fn.store(encode, std::memory_order_release);
  }
  const cuuint32_t estr[2] = {1, 1};
  {
    // packed operands: [rows, K/2] bytes, boxes of 256 rows x 64 bytes, stored unswizzled
    const cuuint64_t pitch4[1] = {(cuuint64_t)(K / 2)};
    const cuuint64_t dim_a4[2] = {(cuuint64_t)(K / 2), (cuuint64_t)M};
    const cuuint64_t dim_b4[2] = {(cuuint64_t)(K / 2), (cuuint64_t)N};
    const cuuint32_t box4[2] = {BK / 2, (cuuint32_t)p.rows_a};
    const cuuint32_t box4b[2] = {BK / 2, (cuuint32_t)(BN / pair)};
    if (encode(&map_a4, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, A.dq4, dim_a4, pitch4, box4, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
    if (encode(&map_b4, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, W.wq4, dim_b4, pitch4, box4b, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }
  p.SS = 0;
  if (stma && !a8) {
    const cuuint64_t pitch[1] = {(cuuint64_t)GK};
    const cuuint64_t dim_a[2] = {(cuuint64_t)GK, (cuuint64_t)M};
    const cuuint64_t dim_b[2] = {(cuuint64_t)GK, (cuuint64_t)N};
    const cuuint32_t box_a[2] = {BK, (cuuint32_t)p.rows_a};
    const cuuint32_t box_b[2] = {BK, (cuuint32_t)(BN / pair)};
    if (encode(&map_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(A.vals), dim_a, pitch, box_a, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
    if (encode(&map_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, W.w_sparse, dim_b, pitch, box_b, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
    p.SS = (int)((GK + BK - 1) / BK);
  }

  if (a8) {
    // the merged 8-bit activations: written once (by expand_a8_kernel here, or by the caller's
    // encode already), read by TMA as [M, K] bytes
    uint8_t* a8buf = static_cast<uint8_t*>(workspace);
    if (!a8_ready) {
      err = launch_expand_a8(b, k, A, positions, M, K, a8buf, st);
      if (err != cudaSuccess) return err;
    }
    const cuuint64_t pitch[1] = {(cuuint64_t)K};
    const cuuint64_t dim_a[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint32_t box_a[2] = {BK, 2 * BM};
    if (encode(&map_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, a8buf, dim_a, pitch, box_a, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
    // `out` as [M, N] bf16 for the epilogue's TMA stores: blocks of 32 rows x 32 columns (64 bytes)
    const cuuint64_t pitch_o[1] = {(cuuint64_t)N * 2};
    const cuuint64_t dim_o[2] = {(cuuint64_t)N, (cuuint64_t)M};
    const cuuint32_t box_o[2] = {32, 32};
    if (encode(&map_b, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, out, dim_o, pitch_o, box_o, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }

#define SQ_LAUNCH_GEMM(PAIR_, MODE_, SPLIT_)                                                                \
  do {                                                                                                      \
    static std::atomic<bool> attr_set_[64]; /* once per kernel variant and device */                       \
    if (!attr_set_[dev].load(std::memory_order_acquire)) {                                                  \
      std::lock_guard<std::mutex> lock_(setup_mutex());                                                     \
      err = cudaFuncSetAttribute(gemm_kernel<PAIR_, MODE_, SPLIT_>,                                         \
                                 cudaFuncAttributeMaxDynamicSharedMemorySize,                               \
                                 Geo<PAIR_, MODE_>::kSmemBytes);                                            \
      if (err != cudaSuccess) return err;                                                                   \
      attr_set_[dev].store(true, std::memory_order_release);                                                \
    }                                                                                                       \
    cudaLaunchConfig_t lc;                                                                                  \
    memset(&lc, 0, sizeof(lc));                                                                             \
    cudaLaunchAttribute la[1];                                                                              \
    la[0].id = cudaLaunchAttributeClusterDimension;                                                         \
    la[0].val.clusterDim.x = (unsigned)cluster_x;                                                           \
    la[0].val.clusterDim.y = 1;                                                                             \
    la[0].val.clusterDim.z = 1;                                                                             \
    lc.gridDim = dim3(grid, 1, 1);                                                                          \
    lc.blockDim = dim3(threads_of(MODE_), 1, 1);                                                            \
    lc.dynamicSmemBytes = Geo<PAIR_, MODE_>::kSmemBytes;                                                           \
    lc.stream = st;                                                                                         \
    lc.attrs = la;                                                                                          \
    lc.numAttrs = cluster_x > 1 ? 1 : 0;                                                                    \
    err = cudaLaunchKernelEx(&lc, gemm_kernel<PAIR_, MODE_, SPLIT_>, p, map_a, map_b, map_a4, map_b4);      \
    if (err != cudaSuccess) return err;                                                                     \
  } while (0)
  if (mode == kModeIndep) {
    if (pair == 2) SQ_LAUNCH_GEMM(2, kModeIndep, false);
    else SQ_LAUNCH_GEMM(1, kModeIndep, false);
  } else if (pair == 2) {
    if (mode == kModeA8) SQ_LAUNCH_GEMM(2, kModeA8, false);
    else if (mode == kModeTma) SQ_LAUNCH_GEMM(2, kModeTma, false);
    else if (mode == kModeMergeProd) SQ_LAUNCH_GEMM(2, kModeMergeProd, false);
    else SQ_LAUNCH_GEMM(2, kModeMergeEpi, false);
  } else if (p.splits > 1) {
    if (mode == kModeTma) SQ_LAUNCH_GEMM(1, kModeTma, true);
    else if (mode == kModeMergeProd) SQ_LAUNCH_GEMM(1, kModeMergeProd, true);
    else SQ_LAUNCH_GEMM(1, kModeMergeEpi, true);
  } else {
    if (mode == kModeTma) SQ_LAUNCH_GEMM(1, kModeTma, false);
    else if (mode == kModeMergeProd) SQ_LAUNCH_GEMM(1, kModeMergeProd, false);
    else SQ_LAUNCH_GEMM(1, kModeMergeEpi, false);
  }
#undef SQ_LAUNCH_GEMM
  if (p.splits > 1 && p.ws != nullptr) {
    const int64_t groups = M * (N / 8);
    int64_t blocks = (groups + 255) / 256;
    if (blocks > 8 * (int64_t)sms) blocks = 8 * (int64_t)sms;
    splitk_finish_kernel<<<(unsigned)blocks, 256, 0, st>>>(p.ws, p.splits, (int)M, (int)N, W.colsum, A.s_hi, W.s_w, out,
                                                         acc_out);
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Measurement aid: the rate at which the tensor core itself takes the product's instruction.  One
// CTA per SM issues tcgen05.mma.kind::i8 (128 x 256 x 32, the tiled kernel's instruction) on
// operands that sit in shared memory and are never reloaded, into the two accumulators in turn,
// and does nothing else: no loads, no widening, no epilogue.  Timed by the caller, it gives the
// INT8 rate the tensor pipe sustains at the clocks of that moment -- the denominator a
// tensor-bound kernel can be held against on this GPU.
__global__ void __launch_bounds__(128, 1) int8_peak_kernel(int iters, int* status) {
  extern __shared__ __align__(1024) uint8_t smem_pk[];  // A: 128 rows x 128 B | B: 256 rows x 128 B
  __shared__ uint64_t bar_s;
  __shared__ uint32_t tmem_slot_s;
  __shared__ int abort_s;
  const int tid = threadIdx.x, warp = tid >> 5;
  if ((smem_u32(smem_pk) & 1023u) != 0) {
    if (tid == 0) atomicExch(status, (int)SQ_ERR_CUDA);
    return;
  }
  // (operands of mixed bits rather than zeros, so that the datapath toggles as it does in a real product)
  for (int i = tid; i < (BM + BN) * BK / 16; i += 128) {
    const uint32_t h = (uint32_t)i * 2654435761u;
    reinterpret_cast<uint4*>(smem_pk)[i] = make_uint4(h, h * 2246822519u, h ^ 0x9E3779B9u, ~h * 3266489917u);
  }
  fence_proxy_async_smem();
  const uint32_t bar = smem_u32(&bar_s);
  if (tid == 0) {
    mbar_init(bar, 1);
    abort_s = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc<1>(smem_u32(&tmem_slot_s), 2 * BN);
    tmem_relinquish<1>();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot_s;
  if (tid == 0) {
    const uint64_t da = make_desc(smem_u32(smem_pk)), db = make_desc(smem_u32(smem_pk + BM * BK));
    constexpr uint32_t idesc = make_idesc(false, BM);
    uint32_t phase = 0;
    bool ok = true;
    for (int it = 0; it < iters && ok; ++it) {
#pragma unroll
      for (int kk = 0; kk < BK / 32; ++kk) umma_i8<1>(tmem + (uint32_t)((it & 1) * BN), da + 2 * kk, db + 2 * kk, idesc, 1u);
      if ((it & 63) == 63 || it == iters - 1) {  // a bounded wait every 256 instructions keeps the queue shallow
        umma_commit<1>(bar);
        ok = mbar_wait(bar, phase, &abort_s);
        phase ^= 1u;
      }
    }
    if (!ok) atomicExch(status, (int)SQ_ERR_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc<1>(tmem, 2 * BN);
}

// Launches the probe on every SM; *ops = the INT8 operations (2 per multiply-add) the launch issues.
cudaError_t launch_int8_peak_probe(int iters, double* ops, int* status, cudaStream_t st) {
  int dev = 0, sms = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;
  const int smem = (BM + BN) * BK;
  err = cudaFuncSetAttribute(int8_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (err != cudaSuccess) return err;
  if (ops != nullptr) *ops = 2.0 * BM * BN * BK * (double)iters * (double)sms;
  int8_peak_kernel<<<(unsigned)sms, 128, smem, st>>>(iters, status);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Split-K scratch that nobody has to allocate: a fixed array in the library's device image.
// Every GPU that loads the library holds these 16 MiB until the process exits.
constexpr size_t kStaticScratchBytes = (size_t)16 << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

size_t gemm_static_scratch_bytes() { return kStaticScratchBytes; }

// launch_gemm with the static array as its workspace.  In host code the array's name is only a
// stand-in for the symbol, not a device address, so the address is asked for once per device
// (with that device current) and remembered; the kernels get the pointer like any other.
cudaError_t launch_gemm_static_scratch(int b, int k, const sq_encoded& A, const sq_weights& W,
                                       const uint8_t* positions, int64_t M, int64_t N, int64_t K, uint16_t* out,
                                       int32_t* acc_out, int* status, cudaStream_t st) {
  static std::atomic<void*> scratch_addr[64];
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  void* ptr = scratch_addr[dev].load(std::memory_order_acquire);
  if (ptr == nullptr) {
    err = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (err != cudaSuccess) return err;
    if (ptr == nullptr) return cudaErrorInvalidSymbol;
    scratch_addr[dev].store(ptr, std::memory_order_release);
  }
  return launch_gemm(b, k, false, A, W, positions, M, N, K, out, acc_out, status, ptr, kStaticScratchBytes, false, st);
}

}  // namespace sq
