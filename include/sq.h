/*
 * sq.h -- C ABI of the B200 (sm_100a) SQ-format library.
 *
 * SQ-format (arXiv 2512.05409, Section 3.1, Eq. 1) stores one GEMM operand as
 * banks of b consecutive elements in which a fixed number k = (1-s)*b of entries
 * is kept in a high precision h_high and the rest in a low precision h_low, plus
 * scales and a mask.  This library implements the setting the paper runs on GPUs
 * (Section 4.1: h_high = INT8, h_low = INT4) for ACTIVATIONS in SQ-format times
 * INT4 per-output-channel weights:
 *
 *     sq_calib_positions   static mask from a calibration batch  (Algorithm 2)
 *     sq_pack_weights      INT4 weights (+ the Alg. 2 row reorder for static masks)
 *     sq_encode            bf16 activations -> SQ-format         (Sections 3.2.2, 3.3)
 *     sq_gemm              dense INT4 + sparse INT8 products, one int32 accumulator,
 *                          one dequantising epilogue             (Section 3.3, Fig. 2b)
 *     sq_decode            SQ-format -> bf16                     (inverse of Eq. 1)
 *
 * Conventions shared by every call
 *   - Tensors are dense and row-major.  Activations X are [M, K] and weights W are
 *     [N, K], both with K contiguous.  Banks run along K: bank g of a row covers
 *     elements g*b .. g*b+b-1, G = K/b banks per row.
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, 16-byte aligned,
 *     sized with sq_encoded_sizes / sq_weights_sizes.  The library allocates nothing
 *     and frees nothing.  The sq_format, sq_encoded and sq_weights structs themselves
 *     live in HOST memory and are read during the call only.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls validate their arguments on the host, enqueue their kernels on that
 *     stream and return without synchronising.  An argument error is reported
 *     synchronously and launches nothing.
 *   - Shape rules: b in {32, 64, 128}; 1 <= k <= b/2; K % 128 == 0 (hence K % b == 0);
 *     K <= SQ_MAX_K; N % 8 == 0; M, N >= 0.  A zero-sized problem (M == 0, or N == 0 for
 *     the weight and GEMM calls) returns SQ_OK right after the shape checks, launches
 *     nothing and does not look at the tensor pointers.
 *   - Inputs are assumed finite.  Rows whose largest magnitude is 0, or lies in
 *     [2^-100, 2^100], are handled exactly; anything else is unspecified.
 *   - Kernels never trap and never spin without bound: a device-side wait that runs
 *     out records SQ_ERR_TIMEOUT in a per-device status word (see sq_device_status)
 *     and the kernel returns after releasing its tensor memory.
 *   - No exceptions, no aborts, no printing.  The library needs an sm_100 device.
 *   - Threads: every call may be made from any host thread, and calls may run concurrently
 *     (the CUDA current device is the calling thread's, as for the CUDA runtime).  The library
 *     keeps per-device host state of two kinds only: first-use caches (device attributes, kernel
 *     attributes, symbol addresses; filled under a lock) and the device status word.  The first
 *     call per device and kernel variant therefore costs more than later ones.  What the library
 *     does NOT arbitrate is the GPU memory the caller passes in: calls that share an output, a
 *     workspace or the static scratch array must be ordered on the GPU by the caller.
 *   - Size limits beyond the shape rules (SQ_ERR_UNSUPPORTED): K <= SQ_MAX_K everywhere; for the
 *     GEMM calls M*K/2, N*K/2 and M*(K/b)*k must each stay below 2^32 bytes and M below 2^23.
 *
 * Number formats (layout version 1)
 *   - INT4 codes are symmetric in [-7, 7] and INT8 codes in [-127, 127]: the most
 *     negative code is never produced (Section 3.2.1).  Two INT4 codes share a byte,
 *     element 2i in the low nibble and 2i+1 in the high nibble, two's complement.
 *   - RNE(p) below is round-half-to-even of the EXACT real product p.
 */
#ifndef SQ_B200_H_
#define SQ_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SQ_LAYOUT_VERSION 1
#define SQ_MAX_K 65536

typedef enum {
  SQ_OK = 0,
  SQ_ERR_INVALID_ARG = 1,  /* a size or format field violates the shape rules      */
  SQ_ERR_UNSUPPORTED = 2,  /* valid in principle but outside what is built (K > SQ_MAX_K) */
  SQ_ERR_NULL_POINTER = 3, /* a required pointer is NULL                            */
  SQ_ERR_ALIGNMENT = 4,    /* a tensor pointer is not 16-byte aligned               */
  SQ_ERR_ARCH = 5,         /* the current device is not sm_100                      */
  SQ_ERR_CUDA = 6,         /* a CUDA runtime call failed (launch, attribute, copy)  */
  SQ_ERR_TIMEOUT = 7       /* a bounded device-side wait expired (sq_device_status) */
} sq_status;

/* How the k positions of a bank are chosen and how the two parts are scaled.
 *   SQ_POS_DYNAMIC       per token, the k largest magnitudes of the bank (Sections 3.2.2, 3.3)
 *   SQ_POS_STATIC        fixed by calibration (Algorithm 2); scales tied: s_lo = s_hi * 2^shift
 *   SQ_POS_STATIC_INDEP  the same positions, but the two parts get independent per-token
 *                        scales as in Algorithm 1 (S_high, S_low): s_hi = (largest selected
 *                        magnitude)/127, s_lo = (largest other magnitude)/7, shift = 0.  sq_gemm
 *                        then keeps two int32 accumulators (dense and sparse product) and joins
 *                        them in fp32: out = bf16(fmaf(acc_hi, s_hi, acc_lo * s_lo) * s_w).
 *                        Needs (K/b)*k to be a multiple of 16 in sq_gemm; with acc_out != NULL
 *                        that buffer holds [2, M, N]: acc_lo first, then acc_hi. */
typedef enum { SQ_POS_DYNAMIC = 0, SQ_POS_STATIC = 1, SQ_POS_STATIC_INDEP = 2 } sq_pos_mode;

/* The part of the Eq. 1 tuple that is a parameter (h_high = INT8, h_low = INT4 fixed). */
typedef struct {
  int32_t bank;     /* b: bank size along K, one of 32, 64, 128                   */
  int32_t k;        /* INT8 entries per bank, k = (1-s)*b, 1 <= k <= b/2          */
  int32_t pos_mode; /* sq_pos_mode: how the k positions of a bank are chosen      */
  int32_t version;  /* SQ_LAYOUT_VERSION                                          */
} sq_format;

/* An activation tensor in SQ-format (device pointers).  G = K/b.
 *   dq4   uint8 [M, K/2]   dense INT4 component, 0 at the bank's k selected positions
 *   vals  int8  [M, G, k]  sparse INT8 component, in ascending bank-local position
 *   idx   uint8 [M, G, k]  bank-local positions (0..b-1) of vals, ascending;
 *                          NULL / unused when pos_mode == SQ_POS_STATIC
 *   s_hi  float [M]        scale of the INT8 component: amax / 127
 *   s_lo  float [M]        scale of the INT4 component: s_hi * 2^shift
 *   shift uint8 [M]        e in 0..4
 * Element j of row m decodes to s_hi*vals at a selected position and s_lo*dq4 elsewhere. */
typedef struct {
  uint8_t* dq4;
  int8_t* vals;
  uint8_t* idx;
  float* s_hi;
  float* s_lo;
  uint8_t* shift;
} sq_encoded;

/* Packed weights (device pointers).
 *   wq4      uint8 [N, K/2]  INT4 codes, per-output-channel symmetric
 *   s_w      float [N]       per-channel scale: wmax / 7
 *   colsum   int32 [N]       sum over K of the channel's INT4 codes
 *   w_sparse int8  [N, G*k]  static masks only: the codes of the selected input
 *                            channels gathered bank by bank (Algorithm 2's reorder) and
 *                            kept in sixteenths, the unit the GEMM's INT8 weight operand
 *                            uses: w_sparse[n, g*k+i] = 16 * code[n, g*b + positions[g][i]];
 *                            NULL / unused when pos_mode == SQ_POS_DYNAMIC */
typedef struct {
  uint8_t* wq4;
  float* s_w;
  int32_t* colsum;
  int8_t* w_sparse;
} sq_weights;

/* Text for a status code (static storage, never NULL). */
const char* sq_status_string(sq_status status);

/* Bytes each member of sq_encoded needs for an [M, K] tensor, in member order
 * (dq4, vals, idx, s_hi, s_lo, shift).  idx is 0 for static positions. */
sq_status sq_encoded_sizes(const sq_format* fmt, int64_t M, int64_t K, size_t bytes_out[6]);

/* Bytes each member of sq_weights needs for [N, K] weights, in member order
 * (wq4, s_w, colsum, w_sparse).  w_sparse is 0 for dynamic positions. */
sq_status sq_weights_sizes(const sq_format* fmt, int64_t N, int64_t K, size_t bytes_out[4]);

/* Static positions (Algorithm 2; Section 3.2.2).  Setup call, not on the timed path.
 *   Abar_j = (sum_t |calib[t,j]|) / T     per-channel mean magnitude, fp64, t ascending
 *   r_j    = sum_n W[n,j]                 signed sum over output channels, fp64, n ascending
 *            (r_j = 1 when W_bf16 is NULL, which ranks by activations alone)
 *   I_j    = |Abar_j * r_j|
 *   positions[g, 0..k) = the k bank-local indices of bank g with the largest I_j
 *                        (equal I_j: smaller j first), stored ascending.
 * calib_bf16: device bf16 [T, K], T >= 1.  W_bf16: device bf16 [N, K] or NULL.
 * positions: device uint8 [K/b, k], written.  fmt->pos_mode must be SQ_POS_STATIC. */
sq_status sq_calib_positions(const sq_format* fmt, const void* calib_bf16, int64_t T, int64_t K,
                             const void* W_bf16, int64_t N, uint8_t* positions, void* cuda_stream);

/* Per-output-channel symmetric INT4 weights (the uniformly quantised operand of
 * Section 3.1 / "classic quantization" of Section 3.2; Algorithm 2's Quant and reorder).
 *   wmax = max_j |W[n,j]|;  code = clamp(RNE(W[n,j] * (7.0f / wmax)), -7, 7);
 *   s_w[n] = wmax / 7.0f (both IEEE fp32 divisions); an all-zero channel gets codes 0, s_w 0.
 * W_bf16: device bf16 [N, K].  positions: device uint8 [K/b, k] for static formats
 * (as written by sq_calib_positions; trusted: distinct, ascending, < b), NULL for
 * dynamic ones.  out: all members written (w_sparse only for static formats). */
sq_status sq_pack_weights(const sq_format* fmt, const void* W_bf16, int64_t N, int64_t K,
                          const uint8_t* positions, sq_weights* out, void* cuda_stream);

/* Activation encode (Sections 3.2.2 and 3.3), per token row m with a_j = X[m,j]:
 *   amax = max_j |a_j|
 *   S    = per bank, the k positions: dynamic -> the k largest |a_j| of the bank
 *          (equal magnitude: smaller j first); static -> positions[g]
 *   rmax = max over j not in S of |a_j|
 *   amax == 0: every code 0, shift 0, s_hi = s_lo = 0.  Otherwise
 *   inv  = 127.0f / amax,  s_hi = amax / 127.0f            (IEEE fp32 divisions)
 *   e    = min{ e in 0..4 : RNE(rmax * inv * 2^-e) <= 7 }, or 4;  s_lo = s_hi * 2^e
 *   j in S:     vals = clamp(RNE(a_j * inv), -127, 127), dense nibble 0
 *   j not in S: dq4  = clamp(RNE(a_j * inv * 2^-e), -7, 7)
 * SQ_POS_STATIC_INDEP (Algorithm 1's separate scales on the static split) instead:
 *   smax = max over j in S of |a_j|;  smax > 0: inv_hi = 127.0f / smax, s_hi = smax / 127.0f
 *   rmax > 0: inv_lo = 7.0f / rmax, s_lo = rmax / 7.0f          (a part that is all zero: 0, 0)
 *   j in S: vals = clamp(RNE(a_j * inv_hi), -127, 127);  else dq4 = clamp(RNE(a_j * inv_lo), -7, 7)
 *   shift = 0
 * X_bf16: device bf16 [M, K].  positions: as for sq_pack_weights.  out: every member
 * written (idx only for dynamic formats). */
sq_status sq_encode(const sq_format* fmt, const void* X_bf16, int64_t M, int64_t K,
                    const uint8_t* positions, sq_encoded* out, void* cuda_stream);

/* Hybrid GEMM (Section 3.3): the dense INT4 product and the sparse INT8 product go
 * into ONE int32 accumulator, followed by one dequantising epilogue:
 *   acc[m,n] = sum_j ( (dq4[m,j] << shift[m]) + [j in S_m] vals[m,j] ) * code[n,j]
 *   out[m,n] = bf16_rne( ((float)acc[m,n] * s_hi[m]) * s_w[n] )
 * SQ_POS_STATIC_INDEP: two accumulators, acc_lo[m,n] = sum_j dq4[m,j] * code[n,j] and
 * acc_hi[m,n] = sum_{j in S} vals[m,j] * code[n,j], joined in fp32:
 *   out[m,n] = bf16_rne( fmaf((float)acc_hi, s_hi[m], (float)acc_lo * s_lo[m]) * s_w[n] )
 * A: an encoding of an [M, K] tensor.  W: packed [N, K] weights of the same format.
 * positions: static formats only (the mask the two were built with), else NULL.
 * out_bf16: device bf16 [M, N], written.  acc_out: device int32 [M, N] or NULL; when
 * given, the raw accumulators are written as well (used by parity tests);
 * SQ_POS_STATIC_INDEP: [2, M, N], acc_lo then acc_hi.
 * Few rows: nothing changes in the result, only in how the work is laid out.
 *   - M <= 32 (and 33 <= M <= 64 while N <= 128 * the number of SMs), K-step selections of 16..64
 *     entries that are a multiple of 16 (static positions: a 16-byte aligned positions array):
 *     a weight-streaming kernel.  The packed weights are the 128-row tensor-core operand (every
 *     SM streams its own slab of output channels), the tokens are the narrow one (16, 32 or 64
 *     accumulator columns), K is cut over
 *     a thread-block cluster whose integer partial sums meet in distributed shared memory.
 *     This kernel is launched with permission to start before its predecessor on the stream has
 *     completed (programmatic dependent launch): until the predecessor has, it reads nothing but
 *     W's packed codes -- its first weight tiles travel while, say, sq_encode of the same tokens
 *     still runs (sq_encode's few-token kernel and this kernel allow their successor that early
 *     start).  So W must not be the output of a kernel that is still running when this call is
 *     made AND that itself releases its successors early; sq_pack_weights does not.
 *   - otherwise M <= 128: K is cut into 2-8 parts that run as one thread-block cluster per tile
 *     of 256 output channels and add their partial sums the same way.
 * Neither needs scratch memory; the result does not depend on the number of parts. */
sq_status sq_gemm(const sq_format* fmt, const sq_encoded* A, const sq_weights* W,
                  const uint8_t* positions, int64_t M, int64_t N, int64_t K, void* out_bf16,
                  int32_t* acc_out, void* cuda_stream);

/* The same product (Section 3.3) with a caller-owned workspace.  The result is bit-identical
 * to sq_gemm's; the workspace only buys speed, in two cases:
 *   - few tokens (M <= 128, decode-shaped): a launch has only N/256 output tiles, each walking
 *     all of K, so most SMs idle.  K is cut into up to 8 parts that run on different SMs,
 *     their raw int32 partial sums go to the workspace ([parts][M][N]) and a second kernel on
 *     the same stream adds them and runs the epilogue;
 *   - more tokens (M > 128, at least four tiles of 256 output channels; dynamic or static
 *     positions): the activations are expanded once into merged 8-bit tensor-core operands
 *     ([M][K] bytes in the workspace) instead of being widened and merged again for every
 *     tile of output channels.
 * SQ_POS_STATIC_INDEP has no use for a workspace (two scales cannot share one merged operand).
 * sq_gemm_workspace_bytes: *bytes = the size this shape and format can make use of, 0 if none
 * (also 0 for the shapes the weight-streaming kernel serves: it needs no scratch).
 * workspace: device memory, 16-byte aligned, or NULL (= sq_gemm); a smaller workspace than
 * asked for is used for fewer parts or not at all, never an error.  Its contents are
 * undefined afterwards; calls that share a workspace must not overlap on the GPU. */
sq_status sq_gemm_workspace_bytes(const sq_format* fmt, int64_t M, int64_t N, int64_t K, size_t* bytes);
sq_status sq_gemm_ws(const sq_format* fmt, const sq_encoded* A, const sq_weights* W,
                     const uint8_t* positions, int64_t M, int64_t N, int64_t K, void* out_bf16,
                     int32_t* acc_out, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Producer fusion (Section 3.3 names fusing the format conversion into the operation that
 * produces the activations; this is the part of it that lies inside the library's boundary):
 * sq_encode that ALSO writes the product's merged 8-bit operand, and the product that reads it.
 *   a8: device uint8 [M, K], 16-byte aligned.  Byte for element j of a row, stored at
 *       32*(j/32) + 16*(j%2) + (j%32)/2 (the tensor-core K order of one 32-element block:
 *       16 even elements, then 16 odd):   j in S: vals + 128,   else: (dq4 << shift) + 128.
 *       It is exactly what sq_gemm_ws writes into an M*K-byte workspace for the same rows.
 *   sq_encode_a8: out as for sq_encode (bit-identical), a8 written in the same call.  Static
 *       positions, tied scales, row lengths that are 8/12/14/16 * 256 * {1,2,4,8}: the encode
 *       kernel writes a8 from the codes it holds in registers; any other format or shape: a
 *       second kernel expands the codes on the same stream.  SQ_POS_STATIC_INDEP:
 *       SQ_ERR_UNSUPPORTED (two scales share no merged operand).
 *   sq_gemm_a8: sq_gemm (bit-identical) reading a8 instead of expanding A again; a8 is never
 *       written.  Shapes the merged operand does not serve (M <= 128, or fewer than four tiles
 *       of 256 output channels) run as sq_gemm and ignore a8.  A, positions: those a8 was
 *       written with. */
sq_status sq_encode_a8(const sq_format* fmt, const void* X_bf16, int64_t M, int64_t K,
                       const uint8_t* positions, sq_encoded* out, void* a8, void* cuda_stream);
sq_status sq_gemm_a8(const sq_format* fmt, const sq_encoded* A, const sq_weights* W,
                     const uint8_t* positions, int64_t M, int64_t N, int64_t K, void* out_bf16,
                     int32_t* acc_out, const void* a8, void* cuda_stream);

/* Producer fusion, the producer itself: the root-mean-square layer normalisation that feeds two
 * of the four quantised linears of the decoder layers whose prefill the appendix "End-to-End
 * Latency Analysis" times, computed inside the encode (static positions, tied scales), so the
 * normalised activation never travels to memory and back.  Per row of X (bf16 [M, K]):
 *     ms = (sum_j x_j^2) / K               in fp64 (every square is exact there)
 *     r  = fp32(1 / sqrt(ms + eps))        one rounding
 *     t  = bf16(fp32(x_j) * r)             fp32 product, round to nearest even
 *     y  = bf16(fp32(t) * fp32(gamma_j))   exact product, one rounding
 * and `out` (and a8, unless NULL) = sq_encode_a8 of y, bit for bit.  gamma_bf16: device bf16
 * [K], 16-byte aligned; eps >= 0.
 *   SQ_POS_STATIC: row lengths that sq_encode_a8's own kernel takes (8/12/14/16 * 256 *
 *     {1,2,4,8}) whose row slots, tables and gamma fit shared memory (K = 4096 and 8192 do, with
 *     or without a8).
 *   SQ_POS_DYNAMIC: k/b in {1/16, 1/8, 1/4, 1/2} (the ratios of sq_encode's fast kernel; the row
 *     is normalised in shared memory before the selection, which then ranks the NORMALISED
 *     magnitudes); a8, if given, is expanded from the codes by a second kernel on the stream.
 *   Anything else, and SQ_POS_STATIC_INDEP: SQ_ERR_UNSUPPORTED, nothing launched (normalise
 *   separately and call sq_encode).  Inputs finite; X is not written. */
sq_status sq_rmsnorm_encode(const sq_format* fmt, const void* X_bf16, const void* gamma_bf16, float eps,
                            int64_t M, int64_t K, const uint8_t* positions, sq_encoded* out, void* a8,
                            void* cuda_stream);

/* (No counterpart in the paper: a convenience of this library.)
 * sq_gemm_ws for callers that have nowhere to get a workspace from.  Some hosts of this
 * library hand out all device memory once, at start-up -- a serving process that gives
 * every component a fixed arena, a plug-in called from someone else's runtime, a plain C
 * caller with no allocator of its own -- and may not call cudaMalloc later: it
 * synchronises the whole device, and it can fail in a process that runs close to full or
 * fragmented memory.  For them the split-K partial sums go into a fixed 16 MiB array that
 * is part of the library's device image (SQ_STATIC_SCRATCH_BYTES; every GPU that loads
 * the library holds it until the process exits).  The call allocates and frees nothing,
 * neither directly nor through any library.
 *   - Inputs, outputs and result are those of sq_gemm (bit-identical).
 *   - Only the few-row case is served: M <= 128 and 2*M*N*4 <= SQ_STATIC_SCRATCH_BYTES
 *     (room for at least two parts of K), otherwise SQ_ERR_UNSUPPORTED and nothing is
 *     launched: call sq_gemm, which needs no scratch.  K is cut into as many parts (2, 4
 *     or 8) as fit the array.
 *   - The first call on each device looks up the array's device address (that device must
 *     be current, as for every call here); make that first call before any stream capture.
 *     The CUDA runtime loads a library's GPU code lazily, so it is also this first call at
 *     which the driver sets the array's 16 MiB aside on that device (unless another call
 *     into the same part of the library has done so before): a host that must know its
 *     memory budget up front makes one call per device during start-up.
 *   - All calls share the one array.  It keeps whatever the previous call left there, which
 *     is harmless: every element a call reads it has written itself first.  But two calls
 *     that overlap on the GPU (different streams, no ordering between them) race on it:
 *     order them, or use sq_gemm_ws with separate workspaces. */
#define SQ_STATIC_SCRATCH_BYTES ((size_t)16 << 20)
sq_status sq_gemm_static_scratch(const sq_format* fmt, const sq_encoded* A, const sq_weights* W,
                                 const uint8_t* positions, int64_t M, int64_t N, int64_t K, void* out_bf16,
                                 int32_t* acc_out, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Floating-point variant: h_high = FP8 (E4M3), h_low = FP4 (E2M1).  Section 3.1 defines the format
 * for floating-point precisions as well; the appendix "FP Quantization Results" uses this pair.
 * The same structs are used with these meanings:
 *   sq_encoded.dq4   uint8 [M, K/2]   dense E2M1 codes (sign, 2 exponent bits, 1 mantissa bit), element
 *                                     2i in the low nibble; code 0 at the bank's k selected positions
 *   sq_encoded.vals  [M, G, k]        sparse E4M3 bytes (OCP FP8: no infinities, largest finite 448)
 *   sq_encoded.idx, s_hi, s_lo, shift as for the integer format; shift e in 0..6
 *   a8               uint8 [M, K]     the MERGED operand the GEMM reads: at a dense place the E4M3 byte of
 *                                     (dense value * 2^e), exact; at a selected place the sparse entry
 *   wq4              uint8 [N, K/2]   E2M1 weight codes;  s_w float [N];  w8 uint8 [N, K]: the same weight
 *                                     values as E4M3 bytes (the GEMM's second operand)
 * Every rounding is to the nearest representable value of the EXACT product, ties to the even
 * code, saturating; a value that rounds to zero is stored as +0.  Per token row, with a_j = X[m,j]:
 *   amax = max_j |a_j|;  amax == 0: every code 0, shift 0, scales 0.  Otherwise
 *   inv = 256.0f / amax, s_hi = amax / 256.0f        (the row maximum maps to 256, not to 448, so
 *                                                     that every dense value times 2^e is an E4M3 number)
 *   S as for sq_encode (dynamic: the k largest |a_j| of the bank, ties to the smaller j; static: positions)
 *   j in S: vals = E4M3(a_j * inv);  rmax = max over j not in S of |a_j|
 *   e = min{ e in 0..6 : rmax * inv * 2^-e <= 6 };  s_lo = s_hi * 2^e;  j not in S: dq4 = E2M1(a_j * inv * 2^-e)
 * Weights, per output channel: wmax = max_j |W[n,j]|, s_w = wmax / 6.0f, code = E2M1(W[n,j] * (6.0f / wmax)).
 * GEMM: acc[m,n] = sum_j value(a8[m,j]) * value(w8[n,j]) on the FP8 tensor-core path with fp32
 * accumulation (the order of the additions is the hardware's), out = bf16_rne((acc * s_hi[m]) * s_w[n]).
 * acc_out: device float [M, N] or NULL.  fmt->pos_mode: SQ_POS_DYNAMIC or SQ_POS_STATIC. */
sq_status sq_fp_pack_weights(const void* W_bf16, int64_t N, int64_t K, uint8_t* wq4, float* s_w, uint8_t* w8,
                             void* cuda_stream);
sq_status sq_fp_encode(const sq_format* fmt, const void* X_bf16, int64_t M, int64_t K, const uint8_t* positions,
                       sq_encoded* out, uint8_t* a8, void* cuda_stream);
/* sq_fp_encode of the output of a root-mean-square layer normalisation, the normalisation computed
 * inside the encode (see sq_rmsnorm_encode: the same definition of y, the same row lengths, static
 * positions only; anything else: SQ_ERR_UNSUPPORTED, nothing launched).  out and a8 = sq_fp_encode
 * of y, bit for bit. */
sq_status sq_fp_rmsnorm_encode(const sq_format* fmt, const void* X_bf16, const void* gamma_bf16, float eps,
                               int64_t M, int64_t K, const uint8_t* positions, sq_encoded* out, uint8_t* a8,
                               void* cuda_stream);
sq_status sq_fp_gemm(const float* s_hi, const uint8_t* a8, const float* s_w, const uint8_t* w8, int64_t M, int64_t N,
                     int64_t K, void* out_bf16, float* acc_out, void* cuda_stream);
sq_status sq_fp_decode(const sq_format* fmt, const sq_encoded* A, const uint8_t* positions, int64_t M, int64_t K,
                       void* out_bf16, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * SQ-format on WEIGHTS: the format part of Algorithm 1 ("SQ-format on Weights") with the storage
 * of Section 3.2.1 and the weight-matrix figure.  Per bank of b input channels of an output
 * channel the k most important weights (importance[n,j] >= 0 is an INPUT: the paper derives it
 * from smoothing and a Hessian of calibration data; equal scores: smaller j first) are kept as
 * INT8 in w_hi [N, K/b, k], compactly and in position order; wq4 [N, K/2] keeps its shape and
 * holds at those places the code the symmetric INT4 range leaves unused (the bit pattern 1000),
 * so the mask is implicit.  Separate per-channel scales (Algorithm 1's S_high, S_low):
 *   s_high[n] = (largest selected |w|) / 127, s_low[n] = (largest other |w|) / 7 (0 for an all-zero part)
 *   w_hi = clamp(RNE(w * (127.0f / hmax)), -127, 127);  wq4 = clamp(RNE(w * (7.0f / lmax)), -7, 7)
 * Storage: K/2 + (K/b)*k bytes per channel = ((1-s)*8 + 4)/8 bytes per weight (Section 4.1's W(SQx)).
 * sq_w_act_quant: per-token symmetric INT8 activations for the product below, s_x = amax / 127,
 *   xq = clamp(RNE(x * (127.0f / amax)), -127, 127); xq [M, K] is written in the order the product
 *   kernel reads it (element j of a group of 8 at byte (j & 1) * 4 + (j >> 1) of the group).
 * sq_w_gemm: the decode-shaped product (weight bytes dominate), M <= 4 tokens, else SQ_ERR_UNSUPPORTED:
 *   acc_lo[m,n] = sum over unmasked j of xq[m,j] * wq4[n,j];  acc_hi[m,n] = sum over masked j of xq[m,j] * w_hi
 *   out[m,n] = bf16_rne( fmaf((float)acc_hi, s_high[n], (float)acc_lo * s_low[n]) * s_x[m] )
 *   acc_out: device int32 [2, M, N] (acc_lo, then acc_hi) or NULL.  Only fmt->bank and fmt->k are used. */
sq_status sq_w_encode(const sq_format* fmt, const void* W_bf16, const float* importance, int64_t N, int64_t K,
                      uint8_t* wq4, int8_t* w_hi, float* s_high, float* s_low, void* cuda_stream);
sq_status sq_w_act_quant(const void* X_bf16, int64_t M, int64_t K, int8_t* xq, float* s_x, void* cuda_stream);
sq_status sq_w_gemm(const sq_format* fmt, const int8_t* xq, const float* s_x, const uint8_t* wq4, const int8_t* w_hi,
                    const float* s_high, const float* s_low, int64_t M, int64_t N, int64_t K, void* out_bf16,
                    int32_t* acc_out, void* cuda_stream);

/* Decode (inverse of Eq. 1): out[m,j] = bf16_rne(s_hi[m]*vals) at selected positions,
 * bf16_rne(s_lo[m]*dq4) elsewhere.  out_bf16: device bf16 [M, K], written. */
sq_status sq_decode(const sq_format* fmt, const sq_encoded* A, const uint8_t* positions,
                    int64_t M, int64_t K, void* out_bf16, void* cuda_stream);

/* Reads and clears the current device's status word.  Synchronises `cuda_stream`
 * first, so every kernel enqueued on it before the call has finished.  Returns
 * SQ_OK, SQ_ERR_TIMEOUT if a kernel gave up on a bounded wait since the last call
 * (its outputs are then undefined), or SQ_ERR_CUDA if the stream reports an error. */
sq_status sq_device_status(void* cuda_stream);

/* Device address of the current device's status word (an int: 0, or the sq_status a kernel
 * recorded), for callers that watch it without synchronising a stream, e.g. with their own
 * asynchronous copy at the end of a batch.  The word belongs to the library; sq_device_status
 * remains the call that clears it.  *device_word is a DEVICE pointer. */
sq_status sq_device_status_word(int** device_word);

/* Measurement aid (the paper has no counterpart): the rate at which this GPU's tensor cores take
 * the product's own instruction.  One CTA per SM issues `iterations` K steps of
 * tcgen05.mma.kind::i8 (128 x 256 x 128 per step) on operands resident in shared memory -- no
 * loads, no widening, no epilogue -- asynchronously on the stream.  *int8_ops (host pointer, may be
 * NULL) receives the number of INT8 operations the launch issues (2 per multiply-add); divided
 * by the launch's device time (CUDA events around the call) it is the INT8 tensor rate a
 * tensor-bound kernel can reach at the clocks of that moment.  1 <= iterations <= 2^24.
 * Uses all of tensor memory on every SM while it runs: not to be overlapped with other calls. */
sq_status sq_probe_int8_tensor_rate(int iterations, double* int8_ops, void* cuda_stream);
/* The same probe for the floating-point variant's instruction (tcgen05.mma.kind::f8f6f4, E4M3 x
 * E4M3, fp32 accumulation): *fp8_ops receives the floating-point operations of the launch. */
sq_status sq_probe_fp8_tensor_rate(int iterations, double* fp8_ops, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SQ_B200_H_ */
