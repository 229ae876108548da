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
// widen, store, proxy fence, arrive: half a microsecond to a microsecond for one group of
// threads, whatever the tile's size), so consecutive K steps are handled by DIFFERENT groups:
//   warp 0      one thread streams the packed tiles of every K step (128 x 64 B of weights,
//               16 x 64 B of activations, the step's sparse values and bank-local indices,
//               16 x nb bytes each) into a ring by TMA
//   warps 1-4   two groups of two warps; group g widens the weights (nibble -> 16 * code, signed)
//               of steps g, g + 2, ... into a ring of three 8-bit stages in the layout the tensor
//               core reads (K-major, 128-byte swizzle)
//   warps 5-8   warp x widens the activation tile (nibble * 2^e + bias, unsigned, offset 128) of
//               steps x, x + 4, ... into a ring of eight small stages of its own and merges the
//               step's sparse INT8 entries into the bytes they belong to
//   warp 9      one thread issues tcgen05.mma.kind::i8 (M = 128 channels, N = 16 tokens) when
//               both operands of a step are ready and hands both stages back
//   warps 10-13 read the accumulator (lane = channel) once the K walk is over
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
constexpr int MT = 16;         // token columns of the accumulator
constexpr int BK = 128;        // K elements per step = bytes per operand row
constexpr int SUP = 1;         // K steps per packed stage (boxes of 4 steps, 256 bytes per row, with one CTA per SM
                               // were measured slower than this with two CTAs per SM)
constexpr int NPK = 4;         // packed stages in flight
constexpr int NW = 3;          // widened weight stages
constexpr int NX = 8;          // widened activation stages
constexpr int kWGroups = 2, kWGroupThreads = 64, kXWarps = 4;
constexpr int kTmaWarp = 0, kFirstW = 1, kFirstX = 5, kMmaWarp = 9, kFirstEpi = 10, kMma2Warp = 14;
constexpr int kThreadsS = 15 * 32;
constexpr int kCtlS = 384 + 2 * SC * 4 + MT * 4;  // barriers, then the slab's constants for the finish
constexpr int kPitch = SUP * (BK / 2);     // bytes per packed row of a stage
constexpr int kPackW = SC * kPitch;        // 32 KB
constexpr int kPackX = MT * kPitch;        // 4 KB
constexpr int kSide = MT * SUP * 64;       // sparse values / indices of a stage: up to 64 per row and step
constexpr int kPackStage = kPackW + kPackX + 2 * kSide;
constexpr int kStageW = SC * BK;           // 16 KB
constexpr int kStageX = MT * BK;           // 2 KB
constexpr int kSmemS = NW * kStageW + NX * kStageX + NPK * kPackStage + kCtlS;
static_assert(kStageX % 1024 == 0 && kPackStage % 128 == 0, "stage alignment");
static_assert(SC * MT * 4 <= NW * kStageW, "partial sums are parked in the weight ring");

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
// D = s32; A (weights, 16 * code) signed; B (activations) unsigned with offset 128; both K-major;
// M = 128, N = 16.
constexpr uint32_t kIdescStream = (2u << 4) | (1u << 7) | (0u << 10) | ((uint32_t)(MT >> 3) << 17) | ((uint32_t)(SC >> 4) << 24);
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}

}  // namespace

__global__ void __launch_bounds__(kThreadsS, 2)
    gemm_stream_kernel(const StreamParams p, const __grid_constant__ CUtensorMap map_w4, const __grid_constant__ CUtensorMap map_x4,
                       const __grid_constant__ CUtensorMap map_sv, const __grid_constant__ CUtensorMap map_si) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = smem_raw;
  if ((smem_u32(smem_raw) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicExch(p.status, (int)SQ_ERR_CUDA);
    return;  // (uniform over the cluster: every CTA sees the same offset of its dynamic block)
  }
  uint8_t* sW = smem;                          // NW x [128 x 128] widened weights
  uint8_t* sX = sW + NW * kStageW;             // NX x [16 x 128] widened (and merged) activations
  uint8_t* sPack = sX + NX * kStageX;          // NPK x [W 128 x 64 | X 16 x 64 | vals 16 x 64 | idx 16 x 64]
  uint8_t* sCtl = sPack + NPK * kPackStage;
  const uint32_t bar_pfull = smem_u32(sCtl);         // NPK: packed stage landed
  const uint32_t bar_pempty = bar_pfull + 8 * NPK;   // NPK: packed stage read by its weight group and activation warp
  const uint32_t bar_wfull = bar_pempty + 8 * NPK;   // NW: weights widened
  const uint32_t bar_wempty = bar_wfull + 8 * NW;    // NW: consumed by the MMAs
  const uint32_t bar_xfull = bar_wempty + 8 * NW;    // NX: activations widened and merged
  const uint32_t bar_xempty = bar_xfull + 8 * NX;    // NX: consumed by the MMAs
  const uint32_t bar_tfull = bar_xempty + 8 * NX;    // accumulator complete
  constexpr int kBars = 2 * NPK + 2 * NW + 2 * NX + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sCtl + 8 * kBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sCtl + 8 * kBars + 8);
  static_assert(8 * kBars + 16 <= 384, "control block too small");
  int32_t* s_cs = reinterpret_cast<int32_t*>(sCtl + 384);   // colsum of the slab's channels
  float* s_sw = reinterpret_cast<float*>(s_cs + SC);        // their weight scales
  float* s_sh = s_sw + SC;                                   // the tokens' scales

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int parts = p.parts;
  const int slab = (int)blockIdx.x / parts, part = (int)blockIdx.x % parts;  // part = rank in the cluster
  const int n0 = slab * SC;
  const int KS = p.KS, k0 = part * KS;
  constexpr uint32_t kTmemCols = 32;

  if (tid == 0) {
    for (int s = 0; s < NPK; ++s) {
      mbar_init(bar_pfull + 8 * s, 1);
      mbar_init(bar_pempty + 8 * s, SUP * (kWGroupThreads + 32));
    }
    for (int s = 0; s < NW; ++s) {
      mbar_init(bar_wfull + 8 * s, kWGroupThreads);
      mbar_init(bar_wempty + 8 * s, 1);
    }
    for (int s = 0; s < NX; ++s) {
      mbar_init(bar_xfull + 8 * s, 32);
      mbar_init(bar_xempty + 8 * s, 1);
    }
    mbar_init(bar_tfull, KS >= 2 ? 2 : 1);  // one arrival per issuing thread that has steps
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kMmaWarp) {
    tmem_alloc<1>(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish<1>();
  }
  if (warp == kTmaWarp && lane == 0) {  // the descriptors are on their way while the barriers are set up
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w4) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x4) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_sv) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_si) : "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == kTmaWarp) {
    // =============================================================== TMA: packed tiles of every K step
    if (lane == 0) {
      const uint32_t bytes = (uint32_t)(kPackW + kPackX + 2 * MT * SUP * p.nb);
      const int nsup = (KS + SUP - 1) / SUP;
      for (int su = 0; su < nsup; ++su) {
        const int ps = su % NPK;
        // (a last stage that holds fewer than SUP steps of this part never completes its "empty"
        // barrier; nothing is loaded after it, so nothing waits for it)
        if (!mbar_wait(bar_pempty + 8 * ps, ((su / NPK) & 1u) ^ 1u, abort_flag)) break;
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
  } else if (warp >= kFirstW && warp < kFirstX) {
    // =============================================================== weights: group g takes steps g, g + 2, ...
    const int wt = tid - kFirstW * 32;            // 0..127
    const int g = wt / kWGroupThreads, gt = wt % kWGroupThreads;
    // thread -> (row % 16, packed 16-byte chunk): a quarter warp reads 128 contiguous packed bytes and
    // its two stores land on eight different 16-byte chunks of the swizzled rows
    const int r16 = gt >> 2, c = gt & 3;
    const uint32_t sw_even = (uint32_t)(((2 * c) ^ (r16 & 7)) << 4);
    bool ok = true;
    for (int ks = g; ks < KS && ok; ks += kWGroups) {
      const int su = ks / SUP, ps = su % NPK, s = ks % NW;
      ok = mbar_wait_park(bar_pfull + 8 * ps, (su / NPK) & 1u, abort_flag);
      if (!ok) break;
      const uint8_t* pk = sPack + ps * kPackStage + r16 * kPitch + (ks % SUP) * 64 + c * 16;
      uint4 rw[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) rw[i] = *reinterpret_cast<const uint4*>(pk + i * 16 * kPitch);  // rows r16 + 16 * i
      ok = mbar_wait_park(bar_wempty + 8 * s, ((ks / NW) & 1u) ^ 1u, abort_flag);
      if (!ok) break;
      uint8_t* w_st = sW + s * kStageW + r16 * 128;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint32_t in[4] = {rw[i].x, rw[i].y, rw[i].z, rw[i].w};
        uint32_t ev[4], od[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          ev[q] = (in[q] << 4) & 0xF0F0F0F0u;
          od[q] = in[q] & 0xF0F0F0F0u;
        }
        uint8_t* dst = w_st + i * 16 * 128;
        *reinterpret_cast<uint4*>(dst + sw_even) = make_uint4(ev[0], ev[1], ev[2], ev[3]);
        *reinterpret_cast<uint4*>(dst + (sw_even ^ 16u)) = make_uint4(od[0], od[1], od[2], od[3]);
      }
      // (only now: every register loaded from the packed stage has been consumed)
      mbar_arrive(bar_pempty + 8 * ps);
      fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor core's async reads
      mbar_arrive(bar_wfull + 8 * s);
    }
  } else if (warp >= kFirstX && warp < kMmaWarp) {
    // =============================================================== activations: warp x takes steps x, x + 4, ...
    const int xw = warp - kFirstX;
    // widening: 64 packed chunks, two per lane: chunk ci = lane + 32 * i -> row ci >> 2, chunk ci & 3
    uint32_t pmul[2], poff[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int row = (lane + 32 * i) >> 2;
      const uint32_t e = row < p.M ? p.shift[row] : 0u;
      pmul[i] = 1u << e;
      poff[i] = 0x01010101u * (128u - (8u << e));
    }
    // merge: two lanes share a row; each takes half of the step's nb entries.  The bank of an entry
    // (and so its K offset inside the step) follows from its index by counting, no division per entry.
    const int mrow = lane >> 1, run = p.nb >> 1, first = (lane & 1) * run;
    const int c_first = first % p.k;
    const uint32_t boff_first = (uint32_t)((first / p.k) * p.b);
    const uint32_t swz = (uint32_t)((mrow & 7) << 4);
    bool ok = true;
    for (int ks = xw; ks < KS && ok; ks += kXWarps) {
      const int su = ks / SUP, ps = su % NPK, sx = ks % NX;
      ok = mbar_wait_park(bar_pfull + 8 * ps, (su / NPK) & 1u, abort_flag);
      if (!ok) break;
      const uint8_t* pk = sPack + ps * kPackStage + kPackW;
      uint4 rx[2];
#pragma unroll
      for (int i = 0; i < 2; ++i)
        rx[i] = *reinterpret_cast<const uint4*>(pk + ((lane + 32 * i) >> 2) * kPitch + (ks % SUP) * 64 + (lane & 3) * 16);
      ok = mbar_wait_park(bar_xempty + 8 * sx, ((ks / NX) & 1u) ^ 1u, abort_flag);
      if (!ok) break;
      uint8_t* x_st = sX + sx * kStageX;
#pragma unroll
      for (int i = 0; i < 2; ++i) {
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
      if (mrow < p.M) {
        const uint8_t* sv = pk + kPackX + mrow * (SUP * p.nb) + (ks % SUP) * p.nb + first;
        const uint8_t* si = sv + kSide;
        uint8_t* xrow = x_st + mrow * 128;
        int cnt = c_first;
        uint32_t boff = boff_first;
        for (int j = 0; j < run; ++j) {
          xrow[(kpos_byte(si[j]) + boff) ^ swz] = (uint8_t)(sv[j] ^ 0x80u);
          if (++cnt == p.k) {
            cnt = 0;
            boff += (uint32_t)p.b;
          }
        }
      }
      mbar_arrive(bar_pempty + 8 * ps);
      fence_proxy_async_smem();
      mbar_arrive(bar_xfull + 8 * sx);
    }
  } else if (warp == kMmaWarp || warp == kMma2Warp) {
    // =============================================================== MMA issuers
    // A K step is four small instructions, but waiting for its two operands, issuing and
    // committing take one thread ~0.5 us: that, not the stream, set the pace of the whole kernel.
    // So TWO threads issue, one the even steps and one the odd ones, each into an accumulator of
    // its own (the sums are integers: the finish adds the two, in any order the same).
    if (lane == 0) {
      const int j = warp == kMmaWarp ? 0 : 1;
      bool ok = true;
      for (int ks = j; ks < KS && ok; ks += 2) {
        const int s = ks % NW, sx = ks % NX;
        ok = mbar_wait(bar_wfull + 8 * s, (ks / NW) & 1u, abort_flag) && mbar_wait(bar_xfull + 8 * sx, (ks / NX) & 1u, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint64_t da = desc_sw128(smem_u32(sW + s * kStageW));
        const uint64_t db = desc_sw128(smem_u32(sX + sx * kStageX));
#pragma unroll
        for (int kk = 0; kk < BK / 32; ++kk)
          umma_i8<1>(tmem + (uint32_t)(j * MT), da + 2 * kk, db + 2 * kk, kIdescStream, (ks > j || kk > 0) ? 1u : 0u);
        umma_commit<1>(bar_wempty + 8 * s);
        umma_commit<1>(bar_xempty + 8 * sx);
      }
      if (ok && j < KS) umma_commit<1>(bar_tfull);
    }
    __syncwarp();
  } else if (warp >= kFirstEpi) {
    // =============================================================== accumulator -> this CTA's partial sums
    // (the rings are idle once the accumulator is complete: every MMA has read its operands)
    const int q = warp & 3;  // a warp reads the tensor-memory lane quarter (warp index mod 4)
    {
      // what the finish needs per channel and token, fetched while the K walk runs
      const int e = tid - kFirstEpi * 32, n = min(n0 + e, p.N - 1);
      s_cs[e] = __ldg(p.colsum + n);
      s_sw[e] = __ldg(p.s_w + n);
      if (e < MT) s_sh[e] = e < p.M ? __ldg(p.s_hi + e) : 0.f;
    }
    if (mbar_wait_idle(bar_tfull, 0, abort_flag)) {
      tc_fence_after();
      const int ch = 32 * q + lane;
      int4* prow = reinterpret_cast<int4*>(smem) + ch * (MT / 4);
      uint32_t v[16];
      tmem_ld16(tmem + ((uint32_t)(32 * q) << 16), v);
      if (KS >= 2) {  // the odd steps' accumulator
        uint32_t v2[16];
        tmem_ld16(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)MT, v2);
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < 16; ++c) v[c] += v2[c];
      }
      tmem_ld_wait();
      // (a warp's 16-byte stores, one 64-byte row per lane, spread over the banks by themselves)
      prow[0] = make_int4((int)v[0], (int)v[1], (int)v[2], (int)v[3]);
      prow[1] = make_int4((int)v[4], (int)v[5], (int)v[6], (int)v[7]);
      prow[2] = make_int4((int)v[8], (int)v[9], (int)v[10], (int)v[11]);
      prow[3] = make_int4((int)v[12], (int)v[13], (int)v[14], (int)v[15]);
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
    const int share = SC / parts, lg = 31 - __clz(share);  // parts is 1, 2, 4 or 8
    for (int i = tid; i < share * p.M; i += kThreadsS) {
      const int ch = part * share + (i & (share - 1)), m = i >> lg;
      const int n = n0 + ch;
      if (n >= p.N) continue;
      const uint32_t laddr = smem_u32(smem) + (uint32_t)(ch * MT + m) * 4u;
      int v = 0;
      if (parts == 1) {
        asm volatile("ld.shared.s32 %0, [%1];" : "=r"(v) : "r"(laddr) : "memory");
      } else {
        // all parts' loads first, then the sum: a load followed by its add would wait out one
        // remote access after the other
        int a[8];
#pragma unroll
        for (int sp = 0; sp < 8; ++sp) {
          a[sp] = 0;
          if (sp < parts)
            asm volatile(
                "{\n\t.reg .b32 ra;\n\t"
                "mapa.shared::cluster.u32 ra, %1, %2;\n\t"
                "ld.shared::cluster.s32 %0, [ra];\n\t}"
                : "=r"(a[sp])
                : "r"(laddr), "r"(sp));
        }
#pragma unroll
        for (int sp = 0; sp < 8; ++sp) v += a[sp];
      }
      const int acc = (v - 2048 * s_cs[ch]) >> 4;
      p.out[(size_t)m * p.N + n] = (uint16_t)f32_to_bf16_bits(((float)acc * s_sh[m]) * s_sw[ch]);
      if (p.acc_out != nullptr) p.acc_out[(size_t)m * p.N + n] = acc;
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
                 uint64_t pitch, uint32_t b0, uint32_t b1, bool swizzle128) {
  constexpr int kSlots = 16;
  thread_local MapKey keys[kSlots];
  thread_local CUtensorMap maps[kSlots];
  thread_local int next = 0;
  const MapKey key{ptr, d0, d1, pitch, b0, b1, swizzle128 ? 1 : 0};
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
             CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
             CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  keys[next] = key;
  maps[next] = *out;
  next = (next + 1) % kSlots;
  return true;
}

cudaError_t launch_stream(const StreamParams& p, const CUtensorMap& mw, const CUtensorMap& mx, const CUtensorMap& msv,
                          const CUtensorMap& msi, int dev, cudaStream_t st) {
  static std::atomic<bool> attr_set[64];
  cudaError_t err;
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(setup_mutex());
    err = cudaFuncSetAttribute(gemm_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemS);
    if (err != cudaSuccess) return err;
    attr_set[dev].store(true, std::memory_order_release);
  }
  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof(lc));
  cudaLaunchAttribute la[1];
  la[0].id = cudaLaunchAttributeClusterDimension;
  la[0].val.clusterDim.x = (unsigned)p.parts;
  la[0].val.clusterDim.y = 1;
  la[0].val.clusterDim.z = 1;
  lc.gridDim = dim3((unsigned)(((p.N + SC - 1) / SC) * p.parts), 1, 1);
  lc.blockDim = dim3(kThreadsS, 1, 1);
  lc.dynamicSmemBytes = kSmemS;
  lc.stream = st;
  lc.attrs = la;
  lc.numAttrs = p.parts > 1 ? 1 : 0;
  return cudaLaunchKernelEx(&lc, gemm_stream_kernel, p, mw, mx, msv, msi);
}

}  // namespace

// Whether launch_gemm_stream takes this call (else the tiled kernel of sq_gemm.cu does).
bool gemm_stream_serves(int b, int k, bool is_static, int64_t M, int64_t K) {
  if (M < 1 || M > MT || is_static) return false;
  const int64_t GK = (K / b) * k;
  const int nb = (BK / b) * k;
  if (GK % 16 != 0) return false;                     // TMA row pitch of vals / idx
  if (nb % 16 != 0 || nb > 64) return false;          // a step's entries travel as one TMA box
  return true;
}

cudaError_t launch_gemm_stream(int b, int k, const sq_encoded& A, const sq_weights& W, const uint8_t* positions, int64_t M,
                               int64_t N, int64_t K, uint16_t* out, int32_t* acc_out, int* status, cudaStream_t st) {
  if (!gemm_stream_serves(b, k, positions != nullptr, M, K)) return cudaErrorNotSupported;
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
  // Parts of K per slab: as many as keep every part at least four K steps long while the launch still
  // fits the GPU in one wave (two CTAs per SM; a cluster's CTAs are co-scheduled).
  const int64_t slabs = (N + SC - 1) / SC, ks = K / BK;
  int parts = 1;
  for (int cand = 2; cand <= 8; cand *= 2) {
    if (ks % cand != 0 || ks / cand < 4 || slabs * cand > 2 * (int64_t)sms) break;
    parts = cand;
  }
  p.parts = parts;
  p.KS = (int)(ks / parts);

  CUtensorMap mw, mx, msv, msi;
  if (!make_map_u8(encode, &mw, W.wq4, (uint64_t)(K / 2), (uint64_t)N, (uint64_t)(K / 2), kPitch, SC, false)) return cudaErrorInvalidValue;
  if (!make_map_u8(encode, &mx, A.dq4, (uint64_t)(K / 2), (uint64_t)M, (uint64_t)(K / 2), kPitch, MT, false)) return cudaErrorInvalidValue;
  if (!make_map_u8(encode, &msv, A.vals, (uint64_t)GK, (uint64_t)M, (uint64_t)GK, (uint32_t)(SUP * nb), MT, false)) return cudaErrorInvalidValue;
  if (!make_map_u8(encode, &msi, A.idx, (uint64_t)GK, (uint64_t)M, (uint64_t)GK, (uint32_t)(SUP * nb), MT, false)) return cudaErrorInvalidValue;
  return launch_stream(p, mw, mx, msv, msi, dev, st);
}

}  // namespace sq
