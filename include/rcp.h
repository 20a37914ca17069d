/*
 * rcp.h -- C ABI of the B200 (sm_100a) library for the decode-time W2A4 hot path of RCP
 * ("Rotate, Clip, and Partition", arXiv 2502.15779).
 *
 * Notation (Section 4.4 of the paper calls the input channels C and the output channels H):
 *   K = input channels, N = output rows, M = tokens (1..16, the decode / skinny regime).
 *
 * Tensor formats (Section 4.4 "Fast GEMV via Latency Hiding", Appendix A.7):
 *   words  uint32 [N][K/16]  2-bit weight codes W_q, 16 per word along K, code 16w+j in bits
 *                            [2j, 2j+1] (least significant first).
 *   lut    fp16   [N][4]     dequantization grid W^_0..W^_3 of Eq. "deqgrid", one per output row.
 *   xq     uint8  [M][K/2]   int4 activations X_q, two per byte: low nibble = even k, high
 *                            nibble = odd k, two's complement.
 *   scale  fp16   [M]        per-token activation scale S.
 *   y      fp16   [M][N]     output O = S * X_q * LUT[W_q].
 *
 * Unless a function says otherwise every pointer is a DEVICE pointer owned by the caller, 16-byte
 * aligned, valid on the current device; `stream` is a cudaStream_t passed as void* (NULL = the
 * default stream). Calls are asynchronous on that stream and allocate no device memory.
 * Every function returns RCP_OK or a negative status; nothing is thrown across this boundary.
 */
#ifndef RCP_H_
#define RCP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  RCP_OK = 0,
  RCP_ERR_NULL = -1,      /* a required pointer is NULL */
  RCP_ERR_SHAPE = -2,     /* K % 64 != 0, N < 1, M outside 1..16, bad had_block, ... */
  RCP_ERR_ALIGN = -3,     /* a pointer is not 16-byte aligned */
  RCP_ERR_CODE = -4,      /* rcp_pack_weights met a code above 3 */
  RCP_ERR_WORKSPACE = -5, /* workspace missing (the streaming kernels report through it) */
  RCP_ERR_CUDA = -6,      /* a CUDA call failed; see rcp_last_cuda_error() */
  RCP_ERR_VARIANT = -7,   /* unknown kernel variant, or the variant does not support the shape */
  RCP_ERR_LIMIT = -8      /* size beyond a fixed capacity of the entry point */
};

/* Text for a status code. Never NULL. */
const char* rcp_status_str(int status);

/* cudaError_t (as int) of the last failed CUDA call made by this library on this thread. */
int rcp_last_cuda_error(void);

/*
 * Weight packing (Section 4.4: W_q is pre-computed offline and stored sub-byte packed along the
 * input channel). codes: uint8 [N][K], each in {0,1,2,3}. words: uint32 [N][K/16].
 * K % 64 == 0. Synchronizes the stream before returning so that RCP_ERR_CODE can be reported;
 * on RCP_ERR_CODE the contents of `words` are unspecified. Calls from several host threads or on several
 * streams may overlap (up to 64 in flight keep separate error flags).
 */
int rcp_pack_weights(const uint8_t* codes, int N, int K, uint32_t* words, void* stream);

/*
 * Per-token activation quantization with the online rotation fused in front
 * (rotation: Section 2.1 / Fig. "rotation", R4 and R_H'; Hadamard matrix: Appendix A.2;
 *  quantizer: Section 4.4 tensor formats, Table "Quantization configurations": symmetric,
 *  per-token, 4 bit).
 *   x_f16      fp16 [M][K] row-major, finite values.
 *   had_block  0 or 1: no rotation. Otherwise a power of two <= 8192 dividing K: every block of
 *              had_block consecutive elements is multiplied by the normalized Sylvester Hadamard
 *              matrix, computed as fp32 butterflies with ascending strides and one final fp32
 *              multiply by 1/sqrt(had_block).
 *   clip_ratio scale = fp16( (max_k |x_rot| * clip_ratio) / 7 ); q = clamp(rne(x_rot/scale),-8,7).
 *              The paper's table uses 0.9; the benchmark configurations use 1.0.
 *   xq, scale  outputs as described at the top. An all-zero token gives scale 0 and q = 0.
 * Constraints: 1 <= M <= 65535, K % 64 == 0, 64 <= K <= 65536.
 */
int rcp_quantize_act(const void* x_f16, int M, int K, int had_block, float clip_ratio,
                     uint8_t* xq, void* scale_f16, void* stream);

/*
 * Kernel variants of the LUT GEMV (all compute the same result).
 *   RCP_GEMV_AUTO    library picks (as measured on B200): DP4A for one token, MMA_ONLY otherwise.
 *   RCP_GEMV_SIMPLE  one warp per output row, scalar decode; also the variant behind S_dbg.
 *   RCP_GEMV_DP4A    streaming kernel, CUDA cores only: masked code planes times int8 activations
 *                    with dp4a, two tokens per launch.
 *   RCP_GEMV_MMA     streaming kernel with the masked code planes as the A operand of int8 mma.sync,
 *                    up to eight tokens per launch (when K is so long that their expanded activations
 *                    would not fit in shared memory at once, the launch goes through K in up to eight
 *                    parts, keeping the integer sums of its rows in shared memory in between; fewer
 *                    tokens per launch only where even that does not fit); nine to sixteen tokens go in one
 *                    launch (two MMA column tiles fed from the same masks) while M * K <= 80 KiB,
 *                    else in launches of eight at most; for one or two tokens the b0*b1
 *                    plane is computed with dp4a beside the tensor cores.
 *   RCP_GEMV_MMA_ONLY  as RCP_GEMV_MMA with all three planes on the tensor cores for every M.
 *   RCP_GEMV_MMA_STREAM  the tensor-core kernel with the expanded activations streamed beside the weights: each
 *                    ring stage carries the int8 activations of the chunks of K its boxes cover, written by a
 *                    warp of its own ahead of the consumers. Nothing is expanded up front, K never has to be
 *                    gone through in parts, and one launch takes up to sixteen tokens whatever K is.
 * The streaming kernel: persistent CTAs, weights through a TMA/mbarrier shared-memory ring, 16-row
 * groups owned by warps, no exchange between CTAs.
 */
enum { RCP_GEMV_AUTO = 0, RCP_GEMV_SIMPLE = 1, RCP_GEMV_DP4A = 2, RCP_GEMV_MMA = 3, RCP_GEMV_MMA_ONLY = 4,
       RCP_GEMV_MMA_STREAM = 5 };

/*
 * Weight-only form of the LUT GEMV (Section 5, the W2-only setting of Table "W2_inference": the codes
 * and the dequantization grid of Section 4.4, activations left in 16-bit floating point):
 *   y[m][n] = sum_k lut[n][ code[n][k] ] * x[m][k]
 * The activations go through the integer kernels as block fixed point (an encoding of this library,
 * the paper has none): per token, with E = floor(log2(max_k |x[m][k]|)), X = round-half-even(x * 2^(21-E))
 * is split into four base-64 digits q0..q3 (q0..q2 in [-32, 31]); each digit plane is one int8 "token" of
 * the tensor-core GEMV, whose exact integer per-code sums are weighted by the grid and the digit's unit
 * 2^(E-21) * 64^d and added in fp32. Elements within 2^-11 of the token's largest magnitude are taken
 * exactly, smaller ones to within 2^(E-22); so |y - exact| <= 2^(E-22) * sum_k |lut[n][code]| plus the
 * fp32 finish and the fp16 rounding of y.
 *   words, lut_f16   DEVICE, as for rcp_gemv_w2a4 (per-row grid).
 *   x_f16            DEVICE fp16 [M][K], finite; 16-byte aligned.
 *   M                1..16 (two tokens per launch, four while 16 * K <= 80 KiB; one token of up to 16384
 *                    elements is split into its digits by the GEMV kernel itself, otherwise a small
 *                    kernel in front does that); K % 64 == 0.
 *   y_f16            DEVICE fp16 [M][N], written.
 *   digits           DEVICE int8 [M][4][K], written: the digit planes (16-byte aligned).
 *   unit             DEVICE fp32 [M][4], written: the unit of each digit plane.
 *   workspace        as for rcp_gemv_w2a4.
 * Asynchronous on `stream`; returns RCP_OK or a negative status.
 */
int rcp_gemv_w2a16(const uint32_t* words, const void* lut_f16, const void* x_f16, int M, int N, int K, void* y_f16,
                   int8_t* digits, float* unit, void* workspace, void* stream);

/*
 * rcp_gemv_w2a16 with the integer sums exported, for parity tests (same section of the paper). S_dbg int32
 * [4 M][N][4]: for digit plane d of token m, entry [4 m + d][n][c] is the sum of that plane's digits over the
 * weights of row n whose code is c, taken from the checked instantiation of the kernel that runs anyway.
 * S_dbg NULL: rcp_gemv_w2a16.
 */
int rcp_gemv_w2a16_checked(const uint32_t* words, const void* lut_f16, const void* x_f16, int M, int N, int K,
                           void* y_f16, int8_t* digits, float* unit, void* workspace, int32_t* S_dbg, void* stream);

/*
 * 3-bit weights (Section 4.3, paragraph "Application of LDP on NF3 format": the paper's other weight setting,
 * W3 in Table "memory" and Table "main_result"): the same look-up-table GEMV with eight levels per quantization
 * unit. The paper prints no storage layout for it; this library's is: the low two bits of a code stored exactly
 * like a 2-bit code, the top bit in a bit plane of its own,
 *   words2  uint32 [N][K/16]  bits [2j, 2j+1] of word w = low two bits of code 16w + j;
 *   words1  uint32 [N][K/32]  word v covers codes 32v .. 32v+31: bit 2i = top bit of code 32v + i,
 *                             bit 2i+1 = top bit of code 32v + 16 + i (i = 0..15),
 * three bits per code in all.
 *
 * rcp_pack_weights3: codes uint8 [N][K], each in 0..7 -> words2, words1. K % 64 == 0. Offline, like
 * rcp_pack_weights: synchronizes the stream to report RCP_ERR_CODE (a code above 7).
 */
int rcp_pack_weights3(const uint8_t* codes, int N, int K, uint32_t* words2, uint32_t* words1, void* stream);

/*
 * W3A4 look-up-table GEMV (Section 4.4 with eight levels):
 *   S_c[m][n][j] = sum over k in group j with code[n][k] == c of q[m][k],  c = 0..7     (exact integers)
 *   y[m][n]      = fp16( scale[m] * sum_j sum_c lut[n][j][c] * S_c[m][n][j] )           (fp32 arithmetic)
 *   lut_f16   DEVICE fp16, 16-byte aligned: [N][8] with group == 0 (one grid per output row), [N][K/128][8] with
 *             group == 128 (one grid per group of 128 weights, the paper's group size); other sizes:
 *             RCP_ERR_SHAPE.
 *   xq, scale_f16, y_f16, M, N, K as for rcp_gemv_w2a4.
 *   S_dbg     NULL in production. Otherwise int32 [M][N][8] ([M][N][K/128][8]) receives S_c from the checked
 *             instantiation of the same kernel.
 * The integer sums are exact (seven sums of q over products of code bits plus the total, turned into the
 * eight S_c by inclusion and exclusion). One token per launch, M launches. Never synchronizes.
 */
int rcp_gemv_w3a4(const uint32_t* words2, const uint32_t* words1, const void* lut_f16, int group,
                  const uint8_t* xq, const void* scale_f16, int M, int N, int K, void* y_f16,
                  int32_t* S_dbg, void* stream);

/*
 * Export of a 3-bit layer trained with a learnable centre to the inputs of rcp_gemv_w3a4 (Section 4.3, paragraph
 * "Application of LDP on NF3 format", Eq. "nf3scales", Eq. "nf3"; clipping range of Section 4.2). Offline, like
 * rcp_ldp_export. A unit is `group` consecutive weights of a row:
 *   lo = sig_beta * min(W), hi = sig_gamma * max(W), h = hi - lo, W clipped to [lo, hi];
 *   c = lo + h * sig_s1 (the centre), s_neg = |c - lo|, s_pos = |hi - c|;
 *   v = (W - c) / s_pos if W > c, else (W - c) / s_neg;
 *   code = index of the table level nearest to v among the levels of v's side (a tie takes the lower level; a
 *          weight equal to c is on the negative side);
 *   level_i = c + table[i] * (s_pos if i > zero_index else s_neg), rounded to fp16.
 * fp32 arithmetic, one rounding per operation. A unit with h <= 0 gets code zero_index and eight levels lo.
 * The paper takes the normalized levels of the format from that format's own publication and prints none, so
 * they are an argument:
 *   table8_host  HOST float [8], strictly ascending, table8_host[zero_index] == 0 (else RCP_ERR_SHAPE); read
 *                during the call.
 *   w_f16, sig_beta, sig_gamma, sig_s1   as for rcp_ldp_export (DEVICE; sigmoids evaluated by the caller).
 *   group      a multiple of 32 dividing K (K for one grid per row).
 *   words2, words1   DEVICE, the layout above; 16-byte aligned.
 *   lut_f16    DEVICE fp16 [N][K/group][8], 16-byte aligned (the lut of rcp_gemv_w3a4 for group 128, or for
 *              group == K with its group argument 0).
 * Never synchronizes; ordering against the GEMV as for rcp_ldp_export.
 */
int rcp_nf3_export(const void* w_f16, const float* sig_beta, const float* sig_gamma, const float* sig_s1,
                   const float* table8_host, int zero_index, int N, int K, int group, uint32_t* words2,
                   uint32_t* words1, void* lut_f16, void* stream);

/*
 * Bytes of caller-provided scratch rcp_gemv_w2a4 needs for this shape (0 on bad shapes). The scratch
 * holds a status word that a kernel sets if one of its bounded waits ever gives up (0 = fine). It
 * must be zero-filled once after allocation; every successful call leaves it zero-filled, so one
 * buffer can serve any sequence of calls.
 */
size_t rcp_gemv_workspace_bytes(int M, int N, int K);

/*
 * Launch plan of the streaming GEMV for a shape, for inspection and tests (host only, touches no
 * GPU). `sms` is the number of CTAs (one per SM; <= 0: 148). Writes up to `cap` ints to `out`:
 *   out[0] tokens per launch, out[1] launches, out[2] ring stages, out[3] shared-memory bytes,
 *   out[4] 128-byte chunks per row, out[5] number of phases, then per phase five ints:
 *   groups per CTA at most, first group, groups in the phase, CTAs taking part, repetitions;
 *   and one last int: the parts of K one launch goes through one after the other (1 unless several tokens
 *   meet a K so long that their expanded activations do not fit in shared memory at once; rcp_gemv_w2a4 then
 *   runs the RCP_GEMV_MMA_STREAM form, one pass over K, where that form's ring fits, and the weight-only form
 *   goes through K in parts).
 * (A group is 16 consecutive output rows; see the kernel's description.) Returns the number of
 * ints the full description has, or a negative status.
 */
int rcp_gemv_plan(int M, int N, int K, int sms, int* out, int cap);

/*
 * LUT GEMV / skinny GEMM (Section 4.4, Eq. "deqgrid"):
 *   S_c[m][n] = sum over k with code[n][k] == c of q[m][k]       (exact integers)
 *   y[m][n]   = fp16( scale[m] * sum_c lut[n][c] * S_c[m][n] )   (fp32 arithmetic)
 * Constraints: 1 <= M <= 16, N >= 1, K % 64 == 0, 64 <= K <= 65536.
 *   workspace  rcp_gemv_workspace_bytes(M,N,K) bytes, see above. Required (RCP_ERR_WORKSPACE without it): every
 *              wait inside the streaming kernels is bounded, and a wait that gives up writes a non-zero code
 *              into its first word (2: the weight producer, 3: a consumer warp) and ends the kernel; the
 *              results of that call are then invalid. Only RCP_GEMV_SIMPLE (no waits) takes NULL.
 *   words, lut_f16 are the constants of the layer: the kernel may start fetching them while earlier
 *              work on the stream is still running (programmatic dependent launch), so that work
 *              must not be writing them. xq, scale, y and workspace obey stream order as usual.
 *   S_dbg      NULL in production. Otherwise int32 [M][N][4] receives S_c, 16-byte aligned; this entry point
 *              then runs the SIMPLE variant. (rcp_gemv_w2a4_variant with a streaming variant and S_dbg runs
 *              the checked instantiation of that very kernel: the same code, which also stores the integer
 *              sums it finishes its rows from. The production instantiations contain no such store.)
 * Never synchronizes.
 */
int rcp_gemv_w2a4(const uint32_t* words, const void* lut_f16, const uint8_t* xq,
                  const void* scale_f16, int M, int N, int K, void* y_f16, void* workspace,
                  int32_t* S_dbg, void* stream);

/* Same, with the kernel variant chosen by the caller (for benchmarks, profiles and the parity tests: with
 * S_dbg set and a variant other than RCP_GEMV_AUTO, S_c comes from the chosen kernel itself). */
int rcp_gemv_w2a4_variant(int variant, const uint32_t* words, const void* lut_f16,
                          const uint8_t* xq, const void* scale_f16, int M, int N, int K,
                          void* y_f16, void* workspace, int32_t* S_dbg, void* stream);

/*
 * Export of a layer trained with learnable direct partitioning to the GEMV's inputs: 2-bit codes,
 * packed, and the four-entry grid of every quantization unit (Section 4.3: Eq. "partition", the
 * equation for t_i, Eq. "quant", Eq. "dequantgrid"; Section 4.4, Eq. "deqgrid"; clipping range of
 * Section 4.2). Offline, like rcp_pack_weights. A unit is `group` consecutive weights of a row:
 *   lo = sig_beta * min(W), hi = sig_gamma * max(W), h = hi - lo, W clipped to [lo, hi];
 *   p1 = sig_s1, p2 = (1 - p1) sig_s2, p3 = (1 - p1)(1 - sig_s2);
 *   t1 = p1/2, t2 = t1 + (p1 + p2)/2, t3 = t2 + (p2 + p3)/2;
 *   code = number of thresholds t_i that (W - lo)/h has reached (equal counts as reached);
 *   levels lo + h * {0, (t1 + t2)/2, (t2 + t3)/2, 1}, rounded to fp16.
 * fp32 arithmetic, one rounding per operation. A unit with h <= 0 gets code 0 and four levels lo.
 *   w_f16      DEVICE fp16 [N][K], the rotated weights; 16-byte aligned.
 *   sig_*      DEVICE float [N][K/group]: the sigmoids of beta, gamma, s_1, s_2, evaluated by the
 *              caller (so that the 2-bit decision does not depend on an exponential's last bit).
 *   group      a multiple of 16 dividing K (K for one grid per row).
 *   words      DEVICE uint32 [N][K/16] (the format of rcp_pack_weights);
 *   lut_f16    DEVICE fp16 [N][K/group][4] (the lut of rcp_gemv_w2a4_grouped; of rcp_gemv_w2a4 when
 *              group == K).
 * Never synchronizes. The GEMV entry points treat words and lut_f16 as constants of the layer and may fetch
 * them before earlier work on their stream has finished (see rcp_gemv_w2a4): let this call complete (stream or
 * event synchronization) before the first GEMV or linear call that reads what it wrote, unless that call is on
 * the same stream directly behind it -- this kernel never signals an early start, so the next kernel on the stream
 * begins only when it has finished.
 */
int rcp_ldp_export(const void* w_f16, const float* sig_beta, const float* sig_gamma,
                   const float* sig_s1, const float* sig_s2, int N, int K, int group,
                   uint32_t* words, void* lut_f16, void* stream);

/*
 * LUT GEMV with one grid per group of weights (Section 4.4: the dequantization grid has shape
 * H x N*4 for N groups per row; Appendix A.3: C = N*G; the table of quantization configurations
 * sets the weight group size G = 128). Weight k of row n takes its levels from lut[n][k / group]:
 *   S_c[m][n][j] = sum over k in [j*group, (j+1)*group) with code[n][k] == c of q[m][k]   (exact)
 *   y[m][n]      = fp16( scale[m] * sum_j sum_c lut[n][j][c] * S_c[m][n][j] )   (fp32 arithmetic;
 *                  the order of the fp32 sum over groups is fixed for a shape, so results repeat)
 *   lut_f16    DEVICE fp16 [N][K/group][4], 8-byte aligned. A constant of the layer like `words`.
 *   group      a multiple of 16 that divides K. group == 128 runs the streaming kernels (up to eight tokens per
 *              launch; where K is so long that their expanded activations do not fit in shared memory, the form
 *              that streams the activations beside the weights); any other size runs the plain kernel
 *              (correct, not tuned).
 *   S_dbg      NULL in production. Otherwise int32 [M][N][K/group][4] receives S_c (plain kernel; through
 *              rcp_gemv_w2a4_grouped_variant with RCP_GEMV_DP4A or RCP_GEMV_MMA_ONLY: the checked
 *              instantiation of that streaming kernel).
 * Everything else as for rcp_gemv_w2a4 (same workspace, same constraints on M, N, K). Returns
 * RCP_ERR_SHAPE for a bad group size. Never synchronizes.
 */
int rcp_gemv_w2a4_grouped(const uint32_t* words, const void* lut_f16, int group, const uint8_t* xq,
                          const void* scale_f16, int M, int N, int K, void* y_f16, void* workspace,
                          int32_t* S_dbg, void* stream);

/* Same, with the kernel variant chosen by the caller: RCP_GEMV_AUTO, RCP_GEMV_SIMPLE,
 * RCP_GEMV_DP4A or RCP_GEMV_MMA_ONLY (the last two want group == 128, else RCP_ERR_VARIANT). */
int rcp_gemv_w2a4_grouped_variant(int variant, const uint32_t* words, const void* lut_f16, int group,
                                  const uint8_t* xq, const void* scale_f16, int M, int N, int K,
                                  void* y_f16, void* workspace, int32_t* S_dbg, void* stream);

/*
 * One decode linear layer from fp16 activations: rcp_quantize_act followed by rcp_gemv_w2a4 (group
 * == 0) or rcp_gemv_w2a4_grouped (group > 0), same arguments, same results bit for bit in xq and
 * scale and within the GEMV's tolerance in y (Section 4.4 data path; Appendix A.7 counts the
 * separate activation quantizer as the overhead this removes).
 *   For one token of 4096 or 8192 elements under one rotation block (had_block == K) and group in
 *   {0, 128}, a single kernel does both: every CTA rotates and quantizes the token itself while its
 *   first weight requests are in flight (measured faster than two kernels for these shapes only).
 *   xq and scale_f16 are then optional outputs (NULL: not written). Every other case runs the two
 *   kernels one after the other and needs xq [M][K/2] and scale_f16 [M] as staging: RCP_ERR_NULL
 *   without them.
 *   x_f16 obeys stream order; words and lut_f16 are layer constants (see rcp_gemv_w2a4).
 * Never synchronizes.
 */
int rcp_linear_w2a4(const void* x_f16, int M, int K, int had_block, float clip_ratio,
                    const uint32_t* words, const void* lut_f16, int group, int N, void* y_f16,
                    uint8_t* xq, void* scale_f16, void* workspace, void* stream);

/*
 * rcp_linear_w2a4 with the exact integer sums exported, for parity tests (Section 4.4: the accumulation has
 * to stay consistent with the grid, and the integer sums S_c are what shows it). Same arguments and results;
 * S_dbg int32 [M][N][4] (group == 0) or [M][N][K/group][4] receives S_c from the checked instantiation of the
 * kernel the call would run anyway (the single kernel with the quantizer inside, or the streaming GEMV behind
 * the stand-alone quantizer; group sizes other than 128 take the plain kernel). S_dbg NULL: rcp_linear_w2a4.
 */
int rcp_linear_w2a4_checked(const void* x_f16, int M, int K, int had_block, float clip_ratio,
                            const uint32_t* words, const void* lut_f16, int group, int N, void* y_f16,
                            uint8_t* xq, void* scale_f16, void* workspace, int32_t* S_dbg, void* stream);

/* Kernel launches one rcp_linear_w2a4 call makes for a shape (1: the single kernel; otherwise the
 * quantizer plus one GEMV launch per batch of tokens). Host only. Negative status on a bad shape. */
int rcp_linear_w2a4_launches(int M, int N, int K, int had_block, int group);

/*
 * One decode linear layer end to end with HOST activations (Section 4.4 data path: rotate and
 * quantize the token, then the LUT GEMV): copies x from host memory, runs rcp_linear_w2a4
 * (per-row grid), copies y back. All on `stream`, no synchronization: y_host is valid after the
 * caller synchronizes the stream. Page-locked (pinned) host buffers are used in place: the quantizer
 * reads x and the GEMV stores y directly in host memory, no copy is made and the staging buffers
 * x_dev / y_dev stay untouched; pageable buffers go through cudaMemcpyAsync and the staging.
 *   x_host_f16  HOST fp16 [M][K];  y_host_f16  HOST fp16 [M][N].
 *   words, lut_f16             DEVICE, the resident packed layer.
 *   x_dev [M][K] fp16, xq_dev [M][K/2], scale_dev [M] fp16, y_dev [M][N] fp16, workspace:
 *                              DEVICE staging owned by the caller (same rules as above).
 */
int rcp_linear_w2a4_host(const void* x_host_f16, int M, int K, int had_block, float clip_ratio,
                         const uint32_t* words, const void* lut_f16, int N, void* y_host_f16,
                         void* x_dev, uint8_t* xq_dev, void* scale_dev, void* y_dev, void* workspace,
                         void* stream);

/*
 * LUT GEMV for callers that cannot allocate device memory. (The paper has no counterpart: this
 * entry point exists for the way the library is embedded, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plug-in inside a serving
 * process whose memory has all been handed to a pool allocator up front, a real-time decode loop
 * that cannot afford the device-wide synchronization an allocation implies, or a host that is
 * already inside a region where allocating calls are forbidden. Such callers can supply inputs
 * and outputs they were given, but not the scratch buffer rcp_gemv_w2a4 asks for.
 *
 * What it does: the same computation as rcp_gemv_w2a4 (variant RCP_GEMV_AUTO, same arguments, same
 * results), with the scratch taken from an array of RCP_STATIC_SCRATCH_BYTES bytes that is part of
 * the library's device image. Every GPU that loads the library holds that array until the process
 * exits. The call makes no cudaMalloc, cudaFree or other allocating call.
 *
 *   - Shapes whose scratch (rcp_gemv_workspace_bytes) exceeds RCP_STATIC_SCRATCH_BYTES are rejected
 *     with RCP_ERR_LIMIT; nothing is launched.
 *   - The first call on each device looks up the array's device address (once per device, with that
 *     device current) and remembers it. Make that first call outside any stream capture.
 *   - The array is shared by every call on the device and keeps whatever the previous call left in
 *     it; each call therefore clears the part it is about to use, on `stream`, before its kernel.
 *   - Because the array is shared, two calls that may overlap on the GPU (different streams, or
 *     different host threads launching concurrently) race on it. Serialize them, or give the
 *     overlapping work to rcp_gemv_w2a4 with scratch buffers of its own.
 * Never synchronizes.
 */
#define RCP_STATIC_SCRATCH_BYTES 4096u
int rcp_gemv_w2a4_static(const uint32_t* words, const void* lut_f16, const uint8_t* xq,
                         const void* scale_f16, int M, int N, int K, void* y_f16, void* stream);

/*
 * The status word of the built-in scratch array (the paper has no counterpart). rcp_gemv_w2a4 callers can look
 * into their own workspace after a call; callers of rcp_gemv_w2a4_static cannot see the array, so this copies
 * its first word to *status_host: 0 = every wait of the calls since the last clearing ended normally, 2 or 3 = a
 * bounded wait gave up (see rcp_gemv_w2a4) and the results of that call are invalid. Synchronizes `stream`;
 * allocates nothing.
 */
int rcp_gemv_w2a4_static_status(int32_t* status_host, void* stream);

/*
 * Self-test of the failure report (a test aid; the paper has no counterpart): launches one thread that waits,
 * with the bounded wait of the GEMV kernels and a limit of `polls` polls (1 .. 2^20), on a barrier nobody
 * arrives at. The wait runs out, the kernel writes code 3 into the first word of `workspace` (NULL: the
 * built-in scratch array of rcp_gemv_w2a4_static) and returns; the context stays usable. Nothing faults and
 * nothing hangs: the limit is the point. Asynchronous on `stream`.
 */
int rcp_selftest_wait_timeout(void* workspace, int polls, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RCP_H_ */
