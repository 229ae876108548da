// Hybrid SQ-format GEMM for a few token rows (at most 16, dynamic positions): bound by the INT4
// weight stream.
//
// Same product as sq_gemm.cu (Section 3.3: dense INT4 part + sparse INT8 part into one int32
// accumulator, one dequantising epilogue), with the operands of the tensor-core instruction
// SWAPPED: the widened weights are the 128-row operand (a CTA owns a slab of 128 output
// channels) and the few tokens are the narrow one (16 columns of the accumulator).  A 128-row
// token tile of which 1 to 16 rows exist would cost the tensor core 8 to 128 times the work per
// weight byte; here an MMA costs 128 x 16 x 32 multiply-adds, so a K step of a slab (8 KB of
// packed weights) is a few dozen cycles of tensor work and the kernel streams weights.
//
// What a K step costs in this shape is not work but hand-over latency (wait for the tile, read,
// widen, store, fence, arrive: a few tenths of a microsecond for one group of threads, whatever
// the tile's size), so consecutive K steps are handled by DIFFERENT groups; and what two CTAs on
// one SM ran out of first was shared-memory bandwidth (a step's 8 KB of packed weights were
// written by TMA, read, written again widened and read by the tensor core: 48 KB), so the widened
// weights -- the MMA's 128-row operand -- now live in TENSOR memory and never pass through shared
// memory a second time:
//   warp 0      one thread streams the packed tiles (boxes of two K steps: 128 x 128 B of weights
//               with the 128-byte swizzle, 16 x 128 B of activations, the steps' sparse values and
//               bank-local indices) into a ring by TMA
//   warps 1-4,  two groups of four warps; group g takes steps g, g + 2, ...  A thread owns one
//   15-18       output channel (tensor-memory lane = quarter warp % 4, lane): it reads the channel's
//               64 packed bytes of the step, widens them (nibble -> 16 * code, signed) and stores
//               them with tcgen05.st into one of six 32-column stages of tensor memory
//   warps 5-8   warp x widens the activation tile (nibble * 2^e + bias, unsigned, offset 128) of
//               steps x, x + 4, ... into a ring of eight small shared-memory stages of its own and
//               merges the step's sparse INT8 entries into the bytes they belong to
//   warps 9,    one thread each issues tcgen05.mma.kind::i8 (A from tensor memory, M = 128
//   14, 19      channels; B from shared memory, N = 16 tokens) for every third step, into an
//               accumulator of its own, and frees both operands' stages with ONE commit per step
//   warps 10-13 read the accumulators (lane = channel) once the K walk is over
//   work item   (slab of 128 output channels, part of K).  The parts of a slab form one
//               thread-block cluster and add their raw int32 partial sums through distributed
//               shared memory; CTA r of the cluster finishes a share of the slab's channels
//               (no scratch memory, no second kernel).  Two CTAs fit an SM.
// Operand encodings, K order inside a 32-element block and the epilogue arithmetic are those of
// sq_gemm.cu, so the int32 sums and the bf16 bits are identical to every other path.  Static
// positions and more than 16 rows stay on the tiled kernel.
// Every wait is bounded; a wait that runs out raises an abort flag, the kernel records
// SQ_ERR_TIMEOUT, and tensor memory is always freed.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <string.h>

#include "sq_device.cuh"
#include "sq_host.h"

namespace sq {

namespace {

constexpr int SC = 128;        // output channels per slab = rows of the MMA = tensor-memory lanes
constexpr int kMaxTokens = 64; // token columns of the accumulator: 16, 32 or 64 (see SG)
constexpr int BK = 128;        // K elements per step = bytes per operand row
constexpr int SUP = 2;         // K steps per packed stage: the TMA engine moves a tile row by row, and 128-byte rows cost it
                               // half of what 64-byte rows do per byte (one step per stage left the weight warps waiting for data)
constexpr int NPK = 4;         // packed stages in flight
constexpr int NW = 6;          // widened weight stages (in tensor memory)
constexpr int kWGroups = 2, kWGroupThreads = 128;
constexpr int kTmaWarp = 0, kFirstW = 1, kFirstX = 5, kMmaWarp = 9, kFirstEpi = 10, kMma2Warp = 14, kFirstW2 = 15, kMma3Warp = 19;
constexpr int kThreadsS = 20 * 32;
constexpr int ND = 24;         // "step done" barriers: a common multiple of NW and NX
constexpr int kCtlBars = 512;
constexpr int kPitch = SUP * (BK / 2);     // bytes per packed row of a stage
constexpr int kPackW = SC * kPitch;        // 16 KB
constexpr int kColsW = BK / 4;              // tensor-memory columns of a widened weight stage (128 lanes x 128 bytes)
// What depends on MT, the token columns of the accumulator (= the N of the MMA).  16 tokens: three
// issuing threads, two CTAs per SM.  32 and 64 tokens: two issuing threads (tensor-memory columns),
// fewer activation stages (shared memory), one CTA per SM.
template <int MT_>
struct SG {
  static constexpr int MT = MT_;
  static constexpr int kIssuers = MT == 16 ? 3 : 2;  // MMA-issuing threads (steps j, j + kIssuers, ... into accumulator j)
  static constexpr int NX = 8;                         // widened activation stages
  // warps that widen and merge activations: four; beyond 16 tokens (their work grows with MT) the four
  // epilogue warps, idle during the K walk, make it eight
  static constexpr int kXWarps = MT == 16 ? 4 : 8;
  static constexpr int kCtlS = kCtlBars + 2 * SC * 4 + MT * 4;  // barriers, then the slab's constants for the finish
  static constexpr int kPackX = MT * kPitch;        // packed activations of a stage
  static constexpr int kSide = MT * SUP * 64;       // sparse values / indices of a stage: up to 64 per row and step
  static constexpr int kPackStage = kPackW + kPackX + 2 * kSide;
  static constexpr int kAccCols = kIssuers * MT;    // one accumulator per issuing thread
  static constexpr int kStageX = MT * BK;
  static constexpr int kSmemS = NX * kStageX + NPK * kPackStage + kCtlS;
  static constexpr uint32_t kTmemCols = kAccCols + NW * kColsW <= 256 ? 256u : 512u;
  static constexpr int kCtasPerSm = MT == 16 ? 2 : 1;
  // D = s32; A (weights, 16 * code) signed; B (activations) unsigned with offset 128; both K-major; M = 128, N = MT
  static constexpr uint32_t kIdesc = (2u << 4) | (1u << 7) | (0u << 10) | ((uint32_t)(MT >> 3) << 17) | ((uint32_t)(SC >> 4) << 24);
  static_assert(kStageX % 1024 == 0 && kPackStage % 1024 == 0 && (NX * kStageX) % 1024 == 0 && SUP <= 2, "stage alignment (swizzled weight tiles)");
  static_assert(SC * MT * 4 <= NPK * kPackStage, "partial sums are parked in the packed ring");
  static_assert(ND % NX == 0 && kAccCols + NW * kColsW <= 512 && kSmemS <= 227 * 1024, "rings");
};

struct StreamParams {
  const float* s_hi;
  const uint8_t* shift;
  const float* s_w;
  const int32_t* colsum;
  uint16_t* out;
  int32_t* acc_out;
  int* status;
  int M, N, K, b, k;
  int nb;        // sparse entries per row and K step
  int shared_positions;  // static positions: every token's entries sit at the same places (one row of them is loaded)
  int parts;     // parts of K per slab = cluster size
  int KS;        // K steps per part
};

__device__ __forceinline__ uint64_t desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
__device__ __forceinline__ uint32_t kpos_byte(uint32_t jj) {  // position of bank-local element jj in the MMA's K order
  return (jj & 0x60u) | ((jj & 1u) << 4) | ((jj & 31u) >> 1);
}
__device__ __forceinline__ void expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread t of the warp writes lane (base lane + t).
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
      "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]: the 128-row operand is read from tensor memory (lane = row,
// four 8-bit K elements per 32-bit column), the narrow one from shared memory.
__device__ __forceinline__ void umma_i8_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}

// Programmatic dependent launch: this kernel may be started while its predecessor on the stream is
// still running.  Until pdl_wait() returns (the predecessor has completed and its writes are
// visible) it touches nothing a predecessor may have written -- only the weights, which are set up
// long before: their first tiles are on their way while the activations are still being encoded.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

}  // namespace

template <int MT>
__global__ void __launch_bounds__(kThreadsS, SG<MT>::kCtasPerSm)
    gemm_stream_kernel(const StreamParams p, const __grid_constant__ CUtensorMap map_w4, const __grid_constant__ CUtensorMap map_x4,
                       const __grid_constant__ CUtensorMap map_sv, const __grid_constant__ CUtensorMap map_si) {
  using G = SG<MT>;
  constexpr int kIssuers = G::kIssuers, NX = G::NX, kXWarps = G::kXWarps, kPackX = G::kPackX, kSide = G::kSide, kPackStage = G::kPackStage;
  constexpr int kAccCols = G::kAccCols, kStageX = G::kStageX;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = smem_raw;
  if ((smem_u32(smem_raw) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicExch(p.status, (int)SQ_ERR_CUDA);
    return;  // (uniform over the cluster: every CTA sees the same offset of its dynamic block)
  }
  uint8_t* sX = smem;                          // NX x [16 x 128] widened (and merged) activations
  uint8_t* sPack = sX + NX * kStageX;          // NPK x [W 128 x 64 | X 16 x 64 | vals 16 x 64 | idx 16 x 64]
  uint8_t* sCtl = sPack + NPK * kPackStage;
  const uint32_t bar_pfull = smem_u32(sCtl);         // NPK: packed stage landed
  const uint32_t bar_pempty = bar_pfull + 8 * NPK;   // NPK: packed stage read by its weight group and activation warp
  const uint32_t bar_wfull = bar_pempty + 8 * NPK;   // NW: weights widened
  const uint32_t bar_xfull = bar_wfull + 8 * NW;     // NX: activations widened and merged
  const uint32_t bar_done = bar_xfull + 8 * NX;      // ND: the MMAs of step ks (barrier ks % ND) have read their operands:
                                                     // ONE commit per step frees both the weight and the activation stage
  const uint32_t bar_tfull = bar_done + 8 * ND;      // accumulator complete
  constexpr int kBars = 2 * NPK + NW + NX + ND + 1;
  static_assert(ND % NW == 0, "a step's barrier must not come round before its stages do");
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sCtl + 8 * kBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sCtl + 8 * kBars + 8);
  static_assert(8 * kBars + 16 <= kCtlBars, "control block too small");
  int32_t* s_cs = reinterpret_cast<int32_t*>(sCtl + kCtlBars);   // colsum of the slab's channels
  float* s_sw = reinterpret_cast<float*>(s_cs + SC);        // their weight scales
  float* s_sh = s_sw + SC;                                   // the tokens' scales

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int parts = p.parts;
  const int slab = (int)blockIdx.x / parts, part = (int)blockIdx.x % parts;  // part = rank in the cluster
  const int n0 = slab * SC;
  const int KS = p.KS, k0 = part * KS;
  constexpr uint32_t kTmemCols = G::kTmemCols;  // the accumulators' columns, then NW x 32 columns of widened weights

  if (warp == kTmaWarp) {
    if (lane == 0) {  // the descriptors are on their way while the barriers are set up
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w4) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x4) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_sv) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_si) : "memory");
      *abort_flag = 0;
    }
    // the barriers sit one after another in shared memory: the warp's lanes set them up side by side
    for (int i = lane; i < kBars; i += 32) {
      uint32_t count = 1;                                             // pfull, step done
      if (i >= NPK && i < 2 * NPK) count = SUP * (kWGroupThreads + 32);  // pempty
      else if (i >= 2 * NPK && i < 2 * NPK + NW) count = kWGroupThreads;  // wfull
      else if (i >= 2 * NPK + NW && i < 2 * NPK + NW + NX) count = 32;    // xfull
      else if (i == kBars - 1) count = KS >= kIssuers ? kIssuers : KS;    // tfull: one arrival per issuing thread that has steps
      mbar_init(bar_pfull + 8 * i, count);
    }
    fence_mbar_init();
  }
  if (warp == kMmaWarp) {
    tmem_alloc<1>(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish<1>();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // =============================================================== activations: warp xw of kXWarps takes steps xw, xw + kXWarps, ...
  auto x_role = [&](const int xw) {
    pdl_wait();  // the tokens' shifts below are the predecessor's to write
    // widening: 4 * MT packed chunks, CPL per lane: chunk ci = lane + 32 * i -> row ci >> 2, chunk ci & 3
    constexpr int CPL = MT / 8;
    uint32_t pmul[CPL], poff[CPL];
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
      const int row = (lane + 32 * i) >> 2;
      const uint32_t e = row < p.M ? p.shift[row] : 0u;
      pmul[i] = 1u << e;
      poff[i] = 0x01010101u * (128u - (8u << e));
    }
    // merge: LPR lanes share a row (two for 16 tokens, one otherwise), each takes its share of the
    // step's nb entries; 32 / LPR rows per pass.  The bank of an entry (and so its K offset inside
    // the step) follows from its index by counting, no division per entry.
    constexpr int LPR = MT <= 32 ? 32 / MT : 1, RPP = 32 / LPR;
    const int run = p.nb / LPR, first = (lane % LPR) * run;
    const int c_first = first % p.k;
    const uint32_t boff_first = (uint32_t)((first / p.k) * p.b);
    bool ok = true;
    for (int ks = xw; ks < KS && ok; ks += kXWarps) {
      const int su = ks / SUP, ps = su % NPK, sx = ks % NX;
      ok = mbar_wait_park(bar_pfull + 8 * ps, (su / NPK) & 1u, abort_flag);
      if (!ok) break;
      const uint8_t* pk = sPack + ps * kPackStage + kPackW;
      uint4 rx[CPL];
#pragma unroll
      for (int i = 0; i < CPL; ++i)
        rx[i] = *reinterpret_cast<const uint4*>(pk + ((lane + 32 * i) >> 2) * kPitch + (ks % SUP) * 64 + (lane & 3) * 16);
      if (ks >= NX) ok = mbar_wait_park(bar_done + 8 * ((ks - NX) % ND), ((ks - NX) / ND) & 1u, abort_flag);
      if (!ok) break;
      uint8_t* x_st = sX + sx * kStageX;
#pragma unroll
      for (int i = 0; i < CPL; ++i) {
        const int row = (lane + 32 * i) >> 2, cc = lane & 3;
        const uint32_t in[4] = {rx[i].x, rx[i].y, rx[i].z, rx[i].w};
        uint32_t ev[4], od[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint32_t u = in[q] ^ 0x88888888u;
          ev[q] = (u & 0x0F0F0F0Fu) * pmul[i] + poff[i];
          od[q] = ((u >> 4) & 0x0F0F0F0Fu) * pmul[i] + poff[i];
        }
        const uint32_t se = (uint32_t)(((2 * cc) ^ (row & 7)) << 4);
        uint8_t* dst = x_st + row * 128;
        *reinterpret_cast<uint4*>(dst + se) = make_uint4(ev[0], ev[1], ev[2], ev[3]);
        *reinterpret_cast<uint4*>(dst + (se ^ 16u)) = make_uint4(od[0], od[1], od[2], od[3]);
      }
      __syncwarp();  // the tile is written: its sparse entries now overwrite the (zero) places they belong to
#pragma unroll
      for (int pass = 0; pass < MT / RPP; ++pass) {
        const int mrow = pass * RPP + lane / LPR;
        if (mrow >= p.M) continue;
        const uint32_t swz = (uint32_t)((mrow & 7) << 4);
        const uint8_t* sv = pk + kPackX + mrow * (SUP * p.nb) + (ks % SUP) * p.nb + first;
        // (static positions: the tile of places has one row, shared by all tokens)
        const uint8_t* si = p.shared_positions ? pk + kPackX + kSide + (ks % SUP) * p.nb + first : sv + kSide;
        uint8_t* xrow = x_st + mrow * 128;
        int cnt = c_first;
        uint32_t boff = boff_first;
        // eight entries at a time: their indices and values come with one 8-byte read each (a lane's
        // run starts on an 8-byte boundary: nb is a multiple of 16), and the eight byte stores do
        // not wait for one another
        for (int j0 = 0; j0 < run; j0 += 8) {
          const uint2 iv = *reinterpret_cast<const uint2*>(si + j0);
          const uint2 vv = *reinterpret_cast<const uint2*>(sv + j0);
          const uint32_t vx = vv.x ^ 0x80808080u, vy = vv.y ^ 0x80808080u;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint32_t jj = ((j < 4 ? iv.x : iv.y) >> (8 * (j & 3))) & 0xFFu;
            const uint32_t val = ((j < 4 ? vx : vy) >> (8 * (j & 3))) & 0xFFu;
            xrow[(kpos_byte(jj) + boff) ^ swz] = (uint8_t)val;
            if (++cnt == p.k) {
              cnt = 0;
              boff += (uint32_t)p.b;
            }
          }
        }
      }
      mbar_arrive(bar_pempty + 8 * ps);
      fence_proxy_async_smem();
      mbar_arrive(bar_xfull + 8 * sx);
    }
  };
  if (warp == kTmaWarp) {
    // =============================================================== TMA: packed tiles of every K step
    if (lane == 0) {
      const uint32_t bytes = (uint32_t)(kPackW + kPackX + 2 * MT * SUP * p.nb);
      const int nsup = (KS + SUP - 1) / SUP;
      // the ring's first stages: the weight tiles at once, the activation tiles when the predecessor is done
      const int npre = nsup < NPK ? nsup : NPK;
      for (int su = 0; su < npre; ++su) {
        expect_tx(bar_pfull + 8 * su, bytes);
        tma_2d(smem_u32(sPack + su * kPackStage), &map_w4, (k0 + su * SUP) * (BK / 2), n0, bar_pfull + 8 * su);
      }
      pdl_wait();
      // From here on a successor may be started: whatever it does before its own wait (fetch its first
      // weight tiles) overlaps this kernel, and its wait still covers this kernel's predecessor too.
      pdl_launch_dependents();
      for (int su = 0; su < npre; ++su) {
        const uint32_t dst = smem_u32(sPack + su * kPackStage), bar = bar_pfull + 8 * su;
        const int kx = k0 + su * SUP;
        tma_2d(dst + kPackW, &map_x4, kx * (BK / 2), 0, bar);
        tma_2d(dst + kPackW + kPackX, &map_sv, kx * p.nb, 0, bar);
        tma_2d(dst + kPackW + kPackX + kSide, &map_si, kx * p.nb, 0, bar);
      }
      for (int su = npre; su < nsup; ++su) {
        const int ps = su % NPK;
        // (a last stage that holds fewer than SUP steps of this part never completes its "empty"
        // barrier; nothing is loaded after it, so nothing waits for it)
        if (!mbar_wait_park(bar_pempty + 8 * ps, ((su / NPK) & 1u) ^ 1u, abort_flag)) break;
        const uint32_t dst = smem_u32(sPack + ps * kPackStage), bar = bar_pfull + 8 * ps;
        const int kx = k0 + su * SUP;  // first K step of the stage; columns past K come back as zeros
        expect_tx(bar, bytes);
        tma_2d(dst, &map_w4, kx * (BK / 2), n0, bar);                 // rows past N come back as zeros
        tma_2d(dst + kPackW, &map_x4, kx * (BK / 2), 0, bar);         // rows past M likewise
        tma_2d(dst + kPackW + kPackX, &map_sv, kx * p.nb, 0, bar);
        tma_2d(dst + kPackW + kPackX + kSide, &map_si, kx * p.nb, 0, bar);
      }
    }
    __syncwarp();
  } else if ((warp >= kFirstW && warp < kFirstX) || (warp >= kFirstW2 && warp < kMma3Warp)) {
    // (weights only: nothing here depends on the predecessor)
    // =============================================================== weights: group g takes steps g, g + 2, ...
    // A thread owns one output channel (its tensor-memory lane: quarter warp % 4, lane): it reads the
    // channel's 64 packed bytes of the step (the tile was laid down with the 64-byte swizzle, so the
    // 16-byte reads of eight consecutive rows fall on different banks), widens them (nibble ->
    // 16 * code, signed; [16 even | 16 odd] bytes per 32 elements, the activations' order) and
    // stores them as the MMA's A operand in TENSOR memory: the 8-bit weights never pass through
    // shared memory, whose bandwidth two CTAs per SM had used up.
    const int g = warp >= kFirstW2 ? 1 : 0;
    const int row = 32 * (warp & 3) + lane;
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    bool ok = true;
    for (int ks = g; ks < KS && ok; ks += kWGroups) {
      const int su = ks / SUP, ps = su % NPK, s = ks % NW;
      ok = mbar_wait_park(bar_pfull + 8 * ps, (su / NPK) & 1u, abort_flag);
      if (!ok) break;
      const uint8_t* pk = sPack + ps * kPackStage + row * kPitch;
      const uint32_t sz = SUP == 1 ? (uint32_t)((row >> 1) & 3) : (uint32_t)(row & 7);  // 64- / 128-byte swizzle
      const uint32_t c0 = (uint32_t)(ks % SUP) * 4u;
      uint4 rw[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) rw[i] = *reinterpret_cast<const uint4*>(pk + (((c0 + (uint32_t)i) ^ sz) << 4));
      if (ks >= NW) ok = mbar_wait_park(bar_done + 8 * ((ks - NW) % ND), ((ks - NW) / ND) & 1u, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t tdst = tmem + lane_base + (uint32_t)(kAccCols + s * kColsW);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint32_t o[16];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const uint4 v = rw[2 * h + i];
          const uint32_t in[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            o[8 * i + q] = (in[q] << 4) & 0xF0F0F0F0u;
            o[8 * i + 4 + q] = in[q] & 0xF0F0F0F0u;
          }
        }
        tmem_st16(tdst + (uint32_t)(16 * h), o);
      }
      // (only now: every register loaded from the packed stage has been consumed)
      mbar_arrive(bar_pempty + 8 * ps);
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      tc_fence_before();
      mbar_arrive(bar_wfull + 8 * s);
    }
  } else if (warp >= kFirstX && warp < kMmaWarp) {
    x_role(warp - kFirstX);
  } else if (warp == kMmaWarp || warp == kMma2Warp || warp == kMma3Warp) {
    // =============================================================== MMA issuers
    // A K step is four small instructions, but waiting for its two operands, issuing and
    // committing take one thread ~0.5 us: that, not the stream, set the pace of the whole kernel.
    // So THREE threads issue (two for more than 16 tokens), thread j the steps j, j + kIssuers, ..., each
    // into an accumulator of its own (the sums are integers: the finish adds them, in any order the same).
    const int j = warp == kMmaWarp ? 0 : (warp == kMma2Warp ? 1 : 2);
    if (lane == 0 && j < kIssuers) {
      bool ok = true;
      for (int ks = j; ks < KS && ok; ks += kIssuers) {
        const int s = ks % NW, sx = ks % NX;
        ok = mbar_wait_park(bar_wfull + 8 * s, (ks / NW) & 1u, abort_flag) && mbar_wait_park(bar_xfull + 8 * sx, (ks / NX) & 1u, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t ta = tmem + (uint32_t)(kAccCols + s * kColsW);
        const uint64_t db = desc_sw128(smem_u32(sX + sx * kStageX));
#pragma unroll
        for (int kk = 0; kk < BK / 32; ++kk)
          umma_i8_ta(tmem + (uint32_t)(j * MT), ta + 8 * kk, db + 2 * kk, G::kIdesc, (ks > j || kk > 0) ? 1u : 0u);
        umma_commit<1>(bar_done + 8 * (ks % ND));
      }
      if (ok && j < KS) umma_commit<1>(bar_tfull);
    }
    __syncwarp();
  } else if (warp >= kFirstEpi) {
    // =============================================================== accumulator -> this CTA's partial sums
    // (the rings are idle once the accumulator is complete: every MMA has read its operands)
    const int q = warp & 3;  // a warp reads the tensor-memory lane quarter (warp index mod 4)
    pdl_wait();  // the tokens' scales are the predecessor's to write (and `out` may be its to read)
    {
      // what the finish needs per channel and token, fetched while the K walk runs
      const int e = tid - kFirstEpi * 32, n = min(n0 + e, p.N - 1);
      s_cs[e] = __ldg(p.colsum + n);
      s_sw[e] = __ldg(p.s_w + n);
      if (e < MT) s_sh[e] = e < p.M ? __ldg(p.s_hi + e) : 0.f;
    }
    if constexpr (kXWarps == 8) x_role(4 + (warp - kFirstEpi));  // idle until the accumulator is complete otherwise
    if (mbar_wait_idle(bar_tfull, 0, abort_flag)) {
      tc_fence_after();
      const int ch = 32 * q + lane;
      // parked token-major, [MT][SC]: a warp's 32 channels of a token are one 128-byte store, and
      // the finish reads eight channels of a token with two 16-byte loads
      int32_t* pcol = reinterpret_cast<int32_t*>(sPack) + ch;
#pragma unroll
      for (int c16 = 0; c16 < MT / 16; ++c16) {  // sixteen tokens at a time
        uint32_t v[16];
        tmem_ld16(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(16 * c16), v);
#pragma unroll
        for (int j = 1; j < kIssuers; ++j)
          if (KS > j) {  // the other issuing threads' accumulators
            uint32_t v2[16];
            tmem_ld16(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(j * MT + 16 * c16), v2);
            tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 16; ++c) v[c] += v2[c];
          }
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < 16; ++c) pcol[(16 * c16 + c) * SC] = (int)v[c];
      }
    }
    tc_fence_before();
  }

  // Every thread of every CTA of the cluster gets here whatever happened before (an aborted wait
  // only leaves garbage to add), so the cluster barriers cannot be missed by anyone.
  tc_fence_before();
  __syncthreads();
  if (parts > 1) cluster_sync_all();
  {
    // CTA `part` finishes channels [part * SC / parts, (part + 1) * SC / parts) of the slab for all
    // tokens: adds the parts' sums (integer: order-free) and runs the usual epilogue arithmetic.
    // A thread takes eight channels of one token: two 16-byte (remote) reads per part, one 16-byte
    // store of the bf16 outputs (N is a multiple of 8, so a group is inside N or outside).
    const int share = SC / parts, g8s = share >> 3, lg = 31 - __clz(g8s);  // parts is 1, 2 or 4
    for (int i = tid; i < p.M * g8s; i += kThreadsS) {
      const int ch0 = part * share + ((i & (g8s - 1)) << 3), m = i >> lg;
      const int n = n0 + ch0;
      if (n >= p.N) continue;
      const uint32_t laddr = smem_u32(sPack) + (uint32_t)(m * SC + ch0) * 4u;
      int v[8] = {0, 0, 0, 0, 0, 0, 0, 0};
      if (parts == 1) {
        asm volatile("ld.shared.v4.s32 {%0, %1, %2, %3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(laddr) : "memory");
        asm volatile("ld.shared.v4.s32 {%0, %1, %2, %3}, [%4];" : "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]) : "r"(laddr + 16u) : "memory");
      } else {
        // all parts' loads first, then the sums: a load followed by its add would wait out one
        // remote access after the other
        int a[4][8];
#pragma unroll
        for (int sp = 0; sp < 4; ++sp) {
#pragma unroll
          for (int t = 0; t < 8; ++t) a[sp][t] = 0;
          if (sp < parts)
            asm volatile(
                "{\n\t.reg .b32 ra;\n\t"
                "mapa.shared::cluster.u32 ra, %8, %9;\n\t"
                "ld.shared::cluster.v4.s32 {%0, %1, %2, %3}, [ra];\n\t"
                "ld.shared::cluster.v4.s32 {%4, %5, %6, %7}, [ra+16];\n\t}"
                : "=r"(a[sp][0]), "=r"(a[sp][1]), "=r"(a[sp][2]), "=r"(a[sp][3]), "=r"(a[sp][4]), "=r"(a[sp][5]), "=r"(a[sp][6]),
                  "=r"(a[sp][7])
                : "r"(laddr), "r"(sp));
        }
#pragma unroll
        for (int sp = 0; sp < 4; ++sp)
#pragma unroll
          for (int t = 0; t < 8; ++t) v[t] += a[sp][t];
      }
      const float sh = s_sh[m];
      int acc[8];
      uint32_t o[4];
#pragma unroll
      for (int t = 0; t < 8; ++t) acc[t] = (v[t] - 2048 * s_cs[ch0 + t]) >> 4;
#pragma unroll
      for (int t = 0; t < 8; t += 2)
        o[t >> 1] = f32_to_bf16_bits(((float)acc[t] * sh) * s_sw[ch0 + t]) |
                    (f32_to_bf16_bits(((float)acc[t + 1] * sh) * s_sw[ch0 + t + 1]) << 16);
      *reinterpret_cast<uint4*>(p.out + (size_t)m * p.N + n) = make_uint4(o[0], o[1], o[2], o[3]);
      if (p.acc_out != nullptr) {
        int4* dst = reinterpret_cast<int4*>(p.acc_out + (size_t)m * p.N + n);
        dst[0] = make_int4(acc[0], acc[1], acc[2], acc[3]);
        dst[1] = make_int4(acc[4], acc[5], acc[6], acc[7]);
      }
    }
  }
  if (parts > 1) cluster_sync_all();  // nobody leaves while a peer may still read its partial sums
  if (tid == 0 && *abort_flag) atomicExch(p.status, (int)SQ_ERR_TIMEOUT);
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc<1>(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------------------

namespace {

struct MapKey {
  const void* ptr;
  uint64_t d0, d1, pitch;
  uint32_t b0, b1;
  int swizzle;
  bool operator==(const MapKey& o) const {
    return ptr == o.ptr && d0 == o.d0 && d1 == o.d1 && pitch == o.pitch && b0 == o.b0 && b1 == o.b1 && swizzle == o.swizzle;
  }
};

// 2-D byte tensor [d1 rows][d0 bytes], row pitch `pitch`, box b0 x b1.  A few-token call is bound by
// the host's launch path, and encoding a tensor map costs about a microsecond, so the last maps are
// remembered per thread (a map is a pure function of these arguments).
bool make_map_u8(PFN_cuTensorMapEncodeTiled encode, CUtensorMap* out, const void* ptr, uint64_t d0, uint64_t d1,
                 uint64_t pitch, uint32_t b0, uint32_t b1, int swizzle) {
  constexpr int kSlots = 16;
  thread_local MapKey keys[kSlots];
  thread_local CUtensorMap maps[kSlots];
  thread_local int next = 0;
  const MapKey key{ptr, d0, d1, pitch, b0, b1, swizzle};
  for (int i = 0; i < kSlots; ++i)
    if (keys[i].ptr != nullptr && keys[i] == key) {
      *out = maps[i];
      return true;
    }
  const cuuint64_t dims[2] = {d0, d1};
  const cuuint64_t pitches[1] = {pitch};
  const cuuint32_t box[2] = {b0, b1};
  const cuuint32_t estr[2] = {1, 1};
  if (encode(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, pitches, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE,
             swizzle == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : (swizzle == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE),
             CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  keys[next] = key;
  maps[next] = *out;
  next = (next + 1) % kSlots;
  return true;
}

template <int MT>
cudaError_t launch_stream(const StreamParams& p, const CUtensorMap& mw, const CUtensorMap& mx, const CUtensorMap& msv,
                          const CUtensorMap& msi, int dev, cudaStream_t st) {
  static std::atomic<bool> attr_set[64];
  cudaError_t err;
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(setup_mutex());
    err = cudaFuncSetAttribute(gemm_stream_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SG<MT>::kSmemS);
    if (err != cudaSuccess) return err;
    attr_set[dev].store(true, std::memory_order_release);
  }
  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof(lc));
  // attributes: the successor-may-start-early permission always, the cluster shape if K is cut
  cudaLaunchAttribute la[2];
  la[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  la[0].val.programmaticStreamSerializationAllowed = 1;
  la[1].id = cudaLaunchAttributeClusterDimension;
  la[1].val.clusterDim.x = (unsigned)p.parts;
  la[1].val.clusterDim.y = 1;
  la[1].val.clusterDim.z = 1;
  lc.gridDim = dim3((unsigned)(((p.N + SC - 1) / SC) * p.parts), 1, 1);
  lc.blockDim = dim3(kThreadsS, 1, 1);
  lc.dynamicSmemBytes = SG<MT>::kSmemS;
  lc.stream = st;
  lc.attrs = la;
  lc.numAttrs = p.parts > 1 ? 2 : 1;
  return cudaLaunchKernelEx(&lc, gemm_stream_kernel<MT>, p, mw, mx, msv, msi);
}

}  // namespace

// Whether launch_gemm_stream takes this call (else the tiled kernel of sq_gemm.cu does).
bool gemm_stream_serves(int b, int k, bool is_static, int64_t M, int64_t N, int64_t K) {
  (void)is_static;  // static positions: the merge reads one shared row of places instead of a row per token
  if (M < 1 || M > kMaxTokens) return false;
  // 33..64 tokens run one CTA per SM: worth it only while every slab of 128 channels has an SM of its
  // own (measured: 13.0 against 14.2 us at N = K = 4096, but 40 against 37 us at N = 28672)
  if (M > 32) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
    if ((N + SC - 1) / SC > sms) return false;
  }
  const int64_t GK = (K / b) * k;
  const int nb = (BK / b) * k;
  if (GK % 16 != 0) return false;                     // TMA row pitch of vals / idx
  if (nb % 16 != 0 || nb > 64) return false;          // a step's entries travel as one TMA box
  return true;
}

cudaError_t launch_gemm_stream(int b, int k, const sq_encoded& A, const sq_weights& W, const uint8_t* positions, int64_t M,
                               int64_t N, int64_t K, uint16_t* out, int32_t* acc_out, int* status, cudaStream_t st) {
  if (!gemm_stream_serves(b, k, positions != nullptr, M, N, K)) return cudaErrorNotSupported;
  const int64_t GK = (K / b) * k;
  const int nb = (BK / b) * k;

  static std::atomic<int> sm_count_of[64];
  static std::atomic<PFN_cuTensorMapEncodeTiled> encode_fn{nullptr};
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

  StreamParams p;
  p.s_hi = A.s_hi;
  p.shift = A.shift;
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
  p.nb = nb;
  p.shared_positions = positions != nullptr ? 1 : 0;
  // Parts of K per slab: up to four, as long as every part is at least four K steps long and the
  // launch still fits the GPU in one wave (two CTAs per SM; a cluster's CTAs are co-scheduled).
  // (Eight parts were measured slower on every shape: what a part saves in K steps, 0.3 us each,
  // the larger cluster's barriers and the finish's remote reads take back.)
  // Token columns: 16, 32 or 64 (more columns: fewer issuing threads and stages, one CTA per SM).
  const int mt = M <= 16 ? 16 : (M <= 32 ? 32 : 64);
  const int64_t slabs = (N + SC - 1) / SC, ks = K / BK;
  int parts = 1;
  for (int cand = 2; cand <= 4; cand *= 2) {
    if (ks % cand != 0 || ks / cand < 4 || slabs * cand > (mt == 16 ? 2 : 1) * (int64_t)sms) break;
    parts = cand;
  }
  p.parts = parts;
  p.KS = (int)(ks / parts);

  CUtensorMap mw, mx, msv, msi;
  if (!make_map_u8(encode, &mw, W.wq4, (uint64_t)(K / 2), (uint64_t)N, (uint64_t)(K / 2), kPitch, SC, SUP == 1 ? 64 : 128)) return cudaErrorInvalidValue;
  if (!make_map_u8(encode, &mx, A.dq4, (uint64_t)(K / 2), (uint64_t)M, (uint64_t)(K / 2), kPitch, (uint32_t)mt, 0)) return cudaErrorInvalidValue;
  if (!make_map_u8(encode, &msv, A.vals, (uint64_t)GK, (uint64_t)M, (uint64_t)GK, (uint32_t)(SUP * nb), (uint32_t)mt, 0)) return cudaErrorInvalidValue;
  // places: a row per token (dynamic), or the one row of static positions (rows past it come back as zeros, unread)
  if (!make_map_u8(encode, &msi, positions != nullptr ? positions : A.idx, (uint64_t)GK, positions != nullptr ? 1u : (uint64_t)M,
                   (uint64_t)GK, (uint32_t)(SUP * nb), (uint32_t)mt, 0))
    return cudaErrorInvalidValue;
  if (mt == 16) return launch_stream<16>(p, mw, mx, msv, msi, dev, st);
  if (mt == 32) return launch_stream<32>(p, mw, mx, msv, msi, dev, st);
  return launch_stream<64>(p, mw, mx, msv, msi, dev, st);
}

}  // namespace sq
