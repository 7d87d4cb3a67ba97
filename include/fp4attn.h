/*
 * fp4attn — full-FP4 attention forward with Direct-P for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Unless an argument says otherwise every pointer is a DEVICE pointer owned by the
 * caller; the library allocates no device memory.  State kept between calls: cached kernel attributes and
 * the driver entry point of the tensor-map encoder (per process), the tensor maps of each host thread's last
 * few attention calls (host memory, a few KB per thread), and the copy streams and events of
 * fp4attn_attention_host (per device, created on first use); fp4attn_release() drops the last two.  Work is
 * enqueued on the caller's stream and calls return without synchronising.  Errors that the host can detect come back as a non-zero
 * status and nothing is launched; nothing throws, prints or exits.
 *
 * Tensor layouts
 *   x, O          bf16  [B, H, N, d] contiguous
 *   packed Q, K   u8    [B, H, N, d/2]   element 2k in bits 0-3 of byte k, 2k+1 in bits 4-7;
 *                                          a nibble is an E2M1 code  s e1 e0 m
 *   packed V      u8    [B, H, d, N/2]   V is stored TRANSPOSED (key index contiguous) because
 *                                          4-bit tensor-core operands must be contraction-major
 *   scale bytes   u8    per (b, h) a grid of 512-byte atoms.  With r the row (query/key index for
 *                       Q and K, head-dim index for V) and c the scale column (d/32 or d/16 for
 *                       Q and K, N/32 for V), atom (r/128, c/4) starts at
 *                       ((r/128) * ceil(C/4) + c/4) * 512 and holds the byte at
 *                       (r%32)*16 + ((r%128)/32)*4 + c%4.  Rows pad to 128, columns to 4, padding
 *                       bytes are written as zero.  This is the order in which the block-scaled
 *                       tcgen05 instruction reads 128 rows x 4 scale factors.
 *   LSE           f32   [B, H, N], natural logarithm
 *
 * Supported shapes: d in {64, 128}; N a multiple of 128, 128 <= N; B, H >= 1; pointers 16-byte
 * aligned (packed operands and scale buffers 128-byte aligned).  Compute capability 10.0 only.
 */
#ifndef FP4ATTN_H_
#define FP4ATTN_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* fp4attn_stream_t;   /* a cudaStream_t; NULL = legacy default stream */

enum {
  FP4ATTN_OK = 0,
  FP4ATTN_ERR_INVALID_ARG = 1,        /* NULL pointer, non-positive size, unknown enum        */
  FP4ATTN_ERR_UNSUPPORTED_SHAPE = 2,  /* d, N outside the supported set                        */
  FP4ATTN_ERR_UNSUPPORTED_ARCH = 3,   /* current device is not compute capability 10.0        */
  FP4ATTN_ERR_ALIGNMENT = 4,          /* a pointer violates the stated alignment               */
  FP4ATTN_ERR_WORKSPACE = 5,          /* workspace missing or too small                        */
  FP4ATTN_ERR_CUDA = 6,               /* a CUDA runtime / driver call failed                   */
  FP4ATTN_ERR_TIMEOUT = 7,            /* written to *device_status by a kernel whose bounded
                                         wait ran out; never returned synchronously            */
  FP4ATTN_ERR_RANGE = 8               /* written to *device_status by a kernel running with a
                                         fixed row reference when a block exponent or a whole row
                                         fell outside the E8M0 range around it; never returned
                                         synchronously                                          */
};

enum { FP4ATTN_FMT_MXFP4 = 0, FP4ATTN_FMT_NVFP4 = 1 };
enum { FP4ATTN_REFERENCE_RUNNING = 0, FP4ATTN_REFERENCE_FIXED = 1 };
enum { FP4ATTN_ROLE_Q = 0, FP4ATTN_ROLE_K = 1, FP4ATTN_ROLE_V = 2 };
/* how a normalised score x = y - E_B + log2 6 becomes an E2M1 probability code */
enum { FP4ATTN_PMAP_IDEAL = 0,    /* q = Q_E2M1(2^x)              (Eq. "ideal-code-path"); how 2^x is evaluated
                                     is stated at fp4attn_fwd                                 */
       FP4ATTN_PMAP_AFFINE = 1,   /* q = Q_E2M1(max(0, A x + B))  (Eq. "affine-code-map")  */
       FP4ATTN_PMAP_HYBRID = 2 }; /* per element pair one of the two: the EX2-density control of
                                     Appendix "SM103 launch and EX2 controls"; see exact_pairs     */

/* Human-readable name of a status code (static storage, never NULL). */
const char* fp4attn_status_string(int status);

/* Library version, major*10000 + minor*100 + patch. */
int fp4attn_version(void);

/* Bytes of the packed E2M1 buffer of one operand: B*H*N*d/2.  0 on invalid arguments. */
size_t fp4attn_packed_bytes(int B, int H, int N, int d);

/* Bytes of the scale buffer of one operand, padded to whole 128x4 atoms (layout above).
 * fmt/role decide the scale grid: Q, K: rows N, columns d/32 (MXFP4) or d/16 (NVFP4);
 * V (MXFP4 only): rows d, columns N/32.  0 on invalid arguments. */
size_t fp4attn_scale_bytes(int fmt, int role, int B, int H, int N, int d);

/* Bytes of scratch fp4attn_quantize needs: 0 for MXFP4; for NVFP4 room for the per-block
 * partial maxima of the tensor-wide amax pass. */
size_t fp4attn_quantize_workspace_bytes(int fmt, int role, int B, int H, int N, int d);

/*
 * Operand quantizer (Section "Problem 2", Table "fp4-formats", Eqs. "nv-scale", "mx-scale").
 *
 * MXFP4: every block of 32 values (along d for Q and K; along the key index for V) with maximum
 *   magnitude a stores the E8M0 byte u = clamp(127 + ceil(log2 a), 1, 254) (u = 0 and all codes 0
 *   for an all-zero block) and the codes q = Q_E2M1(6 v / 2^(u-127)), round to nearest, ties to
 *   even; a value is reconstructed as 2^(u-127) * q / 6 (amplitude convention).
 * NVFP4 (Q, K only): every block of 16 values stores the E4M3 byte of
 *   t = fl32(fl32(a_B * G) / 6) (round to nearest even, saturate at 448) and the codes
 *   q = Q_E2M1(fl32(|v| * fl32(G / S_B))) with the sign of v, S_B the decoded byte; S_B = 0
 *   zeroes the block.  G = fl32(2688 / max|x|) over the whole tensor (1 if it is all zero) is
 *   written to *tensor_scale_out (device); reconstruction is S_B * q / G.
 *
 * x_bf16 [B,H,N,d]; packed_out / scales_out sized by the queries above; tensor_scale_out is
 * required for NVFP4 and ignored (may be NULL) for MXFP4; workspace may be NULL when the size
 * query returns 0.  Outputs are fully overwritten (padding included).
 *
 * Inputs are expected to be finite.  A non-finite value never leads to an out-of-range access or
 * an error return (no address depends on the data); under MXFP4 it only affects its own block
 * (amplitude 2^127, its own code saturated at 6); under NVFP4 an infinity reaches every block through G
 * while a NaN may or may not (the tensor maximum is folded with an operation that drops NaNs), and the bytes
 * written are unspecified.  The attention result for such operands is unspecified.
 */
int fp4attn_quantize(const void* x_bf16, int fmt, int role, int B, int H, int N, int d,
                     void* packed_out, void* scales_out, float* tensor_scale_out,
                     void* workspace, size_t workspace_bytes, fp4attn_stream_t stream);

/* Which of the two powers of two that Eq. "mx-scale" allows becomes the amplitude of an MXFP4 block with
 * maximum magnitude a (the paper fixes none; Section "Problem 2" names both neighbours). */
enum { FP4ATTN_QSCALE_CEIL = 0,    /* alpha = 2^ceil(log2 a): the maximum lands in (3, 6], nothing saturates      */
       FP4ATTN_QSCALE_THR16 = 1,   /* alpha = 2^floor(log2(1.6 a)): maxima up to 1.25 alpha saturate at code 6    */
       FP4ATTN_QSCALE_FLOOR = 2,   /* alpha = 2^floor(log2 a): the maximum always saturates at code 6             */
       FP4ATTN_QSCALE_MSE = 3 };   /* per block the better of floor and ceiling: squared error of the 32 codes,
                                      fp32, d_i = 6 v_i/alpha - q_i exact, fl32(d_i^2) added left to right within
                                      groups of eight, groups as (g0 + g1) + (g2 + g3); floor only if strictly
                                      smaller than four times the ceiling's (its units are four times larger)   */

/*
 * MXFP4 operand quantizer with a selectable amplitude rule (Eq. "mx-scale"): as fp4attn_quantize with
 * fmt = FP4ATTN_FMT_MXFP4, except that the E8M0 byte is u = clamp(127 + e, 1, 254) with e the exponent
 * the rule picks, and that codes are q = Q_E2M1(6 v / 2^(u-127)) saturating at +-6.  FP4ATTN_QSCALE_CEIL
 * gives the bytes of fp4attn_quantize.  The decision is taken on the bf16 bit pattern of the block
 * maximum (significand >= 1.25 for the threshold rule), so it is exact.  Same buffers, layouts,
 * alignment and status codes as fp4attn_quantize; no workspace.
 */
int fp4attn_quantize_mxfp4_rule(const void* x_bf16, int role, int scale_rule, int B, int H, int N, int d,
                                void* packed_out, void* scales_out, fp4attn_stream_t stream);

/* Largest tensor fp4attn_quantize_nvfp4_noalloc accepts: 2^27 elements. */
#define FP4ATTN_NOALLOC_MAX_ELEMENTS (1ull << 27)

/*
 * NVFP4 quantizer for callers that cannot allocate device memory.  (The paper has no counterpart;
 * this is a packaging variant of fp4attn_quantize with fmt = FP4ATTN_FMT_NVFP4, same bytes out.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a region whose memory
 * budget is fixed up front, under a framework whose allocator must not be bypassed, or in a
 * latency-critical loop where an allocation would synchronise the device.  fp4attn_quantize asks
 * such callers for a workspace they have no means to provide.
 *
 * What it does instead: the tensor-wide amax pass keeps its per-block partial maxima in a 4 KB
 * array that lives inside the library image (a file-scope __device__ array), so every GPU that
 * loads the library carries those 4 KB until the process exits.  The array is sized for 1024
 * partial maxima of at most 2^17 elements each; tensors with more than
 * FP4ATTN_NOALLOC_MAX_ELEMENTS elements are rejected with FP4ATTN_ERR_WORKSPACE and nothing is
 * launched.  The call performs no cudaMalloc / cudaFree and calls no allocating library routine.
 *
 * The first call on each device looks up the array's device address (once per device, with that
 * device current) before launching; make that first call outside any stream capture.
 * All calls share the one array: its contents are whatever the previous call left (every slot a
 * call reads it has first overwritten, so nothing needs clearing), and two calls whose kernels
 * overlap on the GPU - different streams, or different host threads - race on it.  Serialise them.
 *
 * x_bf16 [B,H,N,d]; role is FP4ATTN_ROLE_Q or FP4ATTN_ROLE_K; packed_out, scales_out and
 * tensor_scale_out as for fp4attn_quantize.
 */
int fp4attn_quantize_nvfp4_noalloc(const void* x_bf16, int role, int B, int H, int N, int d,
                                   void* packed_out, void* scales_out, float* tensor_scale_out,
                                   fp4attn_stream_t stream);

/*
 * NVFP4 quantizer (Q, K) with one encode factor per (batch, head) unit instead of one per tensor (Section
 * "Pass the forward quantization into backward": the forward saves per-head Q-K global factors): unit
 * (b, h) is quantized exactly as fp4attn_quantize would quantize it alone, with
 * G[b*H + h] = fl32(2688 / max|x[b, h]|) (1 for an all-zero unit).  tensor_scale_out receives B*H floats.
 * Pass the operands to fp4attn_fwd with g_per_head = 1.  Units no longer share a scale, so a head with
 * small magnitudes keeps its precision and (batch, head) units stay independent problems.
 * workspace: device scratch of fp4attn_quantize_nvfp4_per_head_workspace_bytes() bytes, 16-byte aligned.
 * Other arguments, layouts and status codes as for fp4attn_quantize.
 */
size_t fp4attn_quantize_nvfp4_per_head_workspace_bytes(int B, int H, int N, int d);
int fp4attn_quantize_nvfp4_per_head(const void* x_bf16, int role, int B, int H, int N, int d,
                                    void* packed_out, void* scales_out, float* tensor_scale_out,
                                    void* workspace, size_t workspace_bytes, fp4attn_stream_t stream);

/* how the integer exponent E_B of a 32-key probability block follows from its maximum y (Eq. "mx-scale"
 * allows either neighbouring power of two as the amplitude) */
enum { FP4ATTN_PSCALE_CEIL = 0,    /* E_B = ceil(max y): nothing saturates                              */
       FP4ATTN_PSCALE_THR16 = 1,   /* E_B = floor(fl32(max y + fl32(log2 1.6))): the block maximum lands in
                                      [3.75, 7.5) code units, values above 6 saturate; lower P error    */
       FP4ATTN_PSCALE_MSE = 2 };   /* per block the better of ceil(max y) and ceil(max y) - 1 by squared error of the
                                      32 represented probabilities: with v = 6 * 2^(y - ceil) the lower exponent wins
                                      iff sum (2v - q(2v))^2 < 4 sum (v - q(v))^2 (fp32 sums over groups of eight keys,
                                      groups as (g0 + g1) + (g2 + g3)); 2^x by ex2.approx, so a block whose two sums
                                      almost tie may take either exponent.  With the ideal map, one NVFP4 factor per
                                      tensor and the one-query schedule only; about twice the conversions per block */

/* how query tiles are assigned to thread blocks (Section "Two-query execution model") */
enum { FP4ATTN_SCHEDULE_ONE_QUERY = 0,   /* one 128-row query tile per thread block: every shape                 */
       FP4ATTN_SCHEDULE_TWO_QUERY = 1 }; /* two query tiles of a head share every K / V stage and run as two
                                            independent chains with an accumulator each.  Exists where tensor
                                            memory holds two accumulators beside the score slots without overlays:
                                            d = 64, N a multiple of 256, noncausal, one NVFP4 factor per tensor;
                                            anything else returns FP4ATTN_ERR_UNSUPPORTED_SHAPE.  Same results, bit
                                            for bit, as FP4ATTN_SCHEDULE_ONE_QUERY                                */

/* format of the probabilities and of V in the second product */
enum { FP4ATTN_PV_MXFP4 = 0,   /* Direct-P: E2M1 codes with E8M0 block scales for P and V (the path of this library)   */
       FP4ATTN_PV_E4M3 = 1 };  /* FP8 P/V (Section "Training stability selects FP8 P/V"): one E4M3 byte per probability
                                  and per value, no block scales; see fp4attn_fwd and fp4attn_quantize_v_e4m3           */

typedef struct {
  const void *q, *k, *v;            /* packed E2M1 (V transposed)                           */
  const void *q_sf, *k_sf, *v_sf;   /* scale atoms                                           */
  const float *q_G, *k_G;           /* device fp32 encode factors; NVFP4 only, else NULL     */
  int qk_fmt;                       /* format of Q and K; P and V are always MXFP4           */
  float softmax_scale;              /* 0 selects 1/sqrt(d)                                   */
  int p_map;                        /* FP4ATTN_PMAP_IDEAL, _AFFINE or _HYBRID                */
  float affine_a, affine_b;         /* classifier constants; affine_a == 0 selects the
                                       paper's generic fit A = 1.50, B = 1.20                */
  int p_scale_rule;                 /* FP4ATTN_PSCALE_CEIL, _THR16 or _MSE                   */
  int causal;                       /* 1: query row i attends keys 0..i only; 0: all keys     */
  int kv_heads;                     /* K and V hold this many heads ([B, kv_heads, N, d]);
                                       H query heads share them in groups of H / kv_heads
                                       (grouped-query attention).  0 selects H               */
  int exact_pairs;                  /* p_map = FP4ATTN_PMAP_HYBRID only: element pair k of every
                                       32-key block (keys 2k, 2k+1) takes the ideal map where bit k
                                       is set, the affine map elsewhere.  Supported patterns:
                                       0x1111, 0x5555, 0x7777 (4, 8, 12 of 16 pairs exact);
                                       noncausal only                                          */
  int g_per_head;                   /* NVFP4 only: 0 - q_G and k_G point to one factor each; 1 - q_G holds
                                       B*H factors and k_G B*kv_heads, one per (batch, head) unit
                                       (fp4attn_quantize_nvfp4_per_head); with the ideal and the
                                       affine map, not with FP4ATTN_PMAP_HYBRID                 */
  int schedule;                     /* FP4ATTN_SCHEDULE_ONE_QUERY (0, default) or _TWO_QUERY */
  int pv_fmt;                       /* FP4ATTN_PV_MXFP4 (0, default) or FP4ATTN_PV_E4M3: then v holds E4M3 bytes of V^T
                                       [B, kv_heads, d, N] from fp4attn_quantize_v_e4m3, v_sf is ignored, v_G is required;
                                       with the ideal map, the ceiling rule and the one-query schedule only          */
  const float* v_G;                 /* FP4ATTN_PV_E4M3: device fp32 encode factors of V, one per (batch, K/V head)    */
  int row_reference;                /* FP4ATTN_REFERENCE_RUNNING (0, default) or FP4ATTN_REFERENCE_FIXED: the row
                                       reference is the constant fixed_reference for every row (see fp4attn_fwd); with
                                       the ideal and the affine map, the ceiling rule, one factor per tensor, the
                                       one-query schedule and FP4ATTN_PV_MXFP4 only                                   */
  int fixed_reference;              /* FP4ATTN_REFERENCE_FIXED: the reference in octaves (log2 units), -1000 .. 1000    */
  const int* seq_len;               /* NULL, or B device integers: batch entry b is a sequence of seq_len[b] tokens
                                       padded to N (see fp4attn_fwd); values are clamped into 1..N.  With the ideal and
                                       the affine map (and with FP4ATTN_PV_E4M3), one-query schedule only            */
} fp4attn_operands;

/*
 * Noncausal attention forward with Direct-P (Sections "Fix 1" and "Fix 2", Algorithm
 * "direct-p-pack", Eqs. "online-recurrence", "represented-probability", "ideal-code-path",
 * "represented-contributions", "represented-output").
 *
 * S = Q K^T runs as a block-scaled FP4 tensor-core product with fp32 accumulation.  With
 * y = fl32(S * c), c = fl32(fl32(log2(e) * softmax_scale) / k), k = 36 for MXFP4 Q,K (two
 * amplitude-convention operands) or fl32(G_q * G_k) for NVFP4, every block of 32 consecutive keys
 * of a query row takes the integer exponent E_B = ceil(max_j y_j), each score maps straight to
 * the E2M1 code q_j = Q_E2M1(2^(y_j - E_B + log2 6)) (p_map = IDEAL; with p_map = AFFINE the paper's
 * classifier q_j = Q_E2M1(max(0, u_j)), u_j = fl32(S_j * fl32(A c) + fl32(A (log2 6 - E_B) + B)), a single
 * fused multiply-add per score, replaces the exponential; with p_map = HYBRID a fixed pattern of element
 * pairs, exact_pairs, keeps the exponential and the rest takes the classifier), and the block's E8M0 byte is
 * E_B - mu + 127 for an integer row reference mu that never exceeds the running maximum by
 * construction (blocks whose byte would drop below 1 are zero blocks).  P V runs as a second
 * block-scaled FP4 product; the output is normalised by the sum of the same rounded values:
 *   O = sum_j p~_j V^_j / sum_j p~_j,   p~_j = 2^(E_B) q_j / 6,   LSE = ln sum_j p~_j.
 *
 * Row reference.  By default (FP4ATTN_REFERENCE_RUNNING) mu follows the running maximum as described, which places no
 * limit on the spread of the logits.  FP4ATTN_REFERENCE_FIXED is the shiftless path of the paper's `fast` policy
 * (Section "Fix 3: guard only extreme model logits"; Table "policy-definition": no anchor): mu is the constant
 * fixed_reference for every row, the softmax warps publish the byte E_B - mu + 127 themselves and nothing is ever
 * rescaled, which takes the row-reference pass out of the chain between the score and the second product.  Codes do
 * not depend on mu, so inside the range the result is that of the running reference (O to the last bit, LSE to float32
 * rounding).  The range: a block whose byte would fall below 1 is a zero block (correct when it lies more than 126
 * octaves below its row's maximum, wrong otherwise); a byte above 254, or a row whose represented sum comes out as 0,
 * cannot be represented - the kernel then writes FP4ATTN_ERR_RANGE to *device_status and the affected rows are
 * unspecified.  With fixed_reference = 0 every row whose largest logit y lies between about -120 and +127 is inside.
 *
 * Range of the logits: |y| < 2^21 is assumed (the block exponent is formed by a float32 rounding trick that is exact
 * there, and block maxima are clamped to that range); inputs whose scaled scores exceed two million octaves lie
 * outside any softmax's useful range and give finite but unspecified results.
 *
 * With causal = 1 (the forward the paper's training section starts from, Section "Causal backward")
 * keys j > i are removed from row i before anything else: they never raise a block maximum, always
 * code to 0, and a block without a visible key contributes nothing.  B, H, N, d describe Q and O;
 * K and V have kv_heads heads.
 *
 * Padded sequences.  With seq_len != NULL, batch entry b holds a sequence of L = seq_len[b] tokens (1 <= L <= N) in
 * buffers laid out for N: keys L..N-1 are removed from every row of that entry exactly as a causal row's invisible
 * keys are (a block's maximum, hence its exponent, is taken over the keys that exist), key tiles that lie entirely
 * beyond L are neither loaded nor multiplied, query tiles that lie entirely beyond L walk one key tile only, and rows
 * L..N-1 of O and LSE receive unspecified finite values.  The quantizers see the padded buffers: MXFP4 rows of Q and K
 * are quantized one by one, so their padding rows only have to be finite; a 32-key block of V that straddles L takes its
 * scale from all 32 keys, and an NVFP4 encode factor from the maximum over the whole tensor (or unit), so V's padding
 * keys and, with NVFP4, all padding should hold zeros unless they are meant to take part in those maxima.  Combines with
 * causal = 1 and with grouped K/V heads.
 *
 * What FP4ATTN_PMAP_IDEAL guarantees.  x is one fused multiply-add in float32, x = fma(S, c, fl32(log2 6 - E_B)).
 * Of the 16 element pairs (keys 2k, 2k+1) of a block, pairs 0, 5, 10 and 15 evaluate 2^x by a degree-6
 * polynomial through the seven points where a code can change (after clamping x at -2.75, below which the
 * code is 0 either way), the other twelve by ex2.approx; the pattern is fixed in this build of the library.
 * Both are monotone there, so the codes equal Q_E2M1(2^x) except for x within about three float32 spacings of
 * a rounding boundary log2(t), t in {1/4, 3/4, 5/4, 7/4, 5/2, 7/2, 5}, where either neighbouring code may come
 * out.  FP4ATTN_PMAP_AFFINE has no such band: its arithmetic is exact float32 as written above.
 *
 * O_bf16 [B,H,N,d]; LSE [B,H,N] (may be NULL); device_status (may be NULL) receives
 * FP4ATTN_ERR_TIMEOUT if a bounded in-kernel wait ran out (or FP4ATTN_ERR_RANGE, see above), and is otherwise left
 * untouched, so the caller clears it beforehand.
 */
int fp4attn_fwd(const fp4attn_operands* ops, int B, int H, int N, int d,
                void* O_bf16, float* LSE, int* device_status, fp4attn_stream_t stream);

/*
 * E4M3 quantizer of V for the FP8 P/V route (Section "Training stability selects FP8 P/V": the retained training
 * route keeps V in E4M3; the paper states no scale rule).  Every (batch, head) unit gets one encode factor
 * G[b*H + h] = fl32(448 / max|V[b, h]|) (1 for an all-zero unit), written to unit_scale_out (B*H floats), and
 * every value the byte Q_E4M3(fl32(v * G)), round to nearest even; a value is reconstructed as decode(byte) / G.
 * bytes_out receives V^T, [B, H, d, N] bytes (key index contiguous: the contraction-major layout of the second
 * product).  workspace: device scratch of fp4attn_quantize_v_e4m3_workspace_bytes() bytes, 16-byte aligned.
 * Shapes, alignment and status codes as for fp4attn_quantize.
 *
 * With pv_fmt = FP4ATTN_PV_E4M3 fp4attn_fwd computes, for FP4 Q and K exactly as described above,
 *   mu_i = ceil(max_j y_ij),  p8_ij = Q_E4M3(2^(y_ij - mu_i + 8)),  O_i = sum_j p8_ij V^_j / sum_j p8_ij,
 *   LSE_i = ln2 (mu_i - 8 + log2 sum_j p8_ij):
 * the row reference is the row's own maximum rounded up to an integer, taken by a first sweep over the keys
 * before any probability is formed (without block scales a rounded probability cannot be re-scaled later), so the
 * result does not depend on any tile order.  2^x is ex2.approx: a byte can differ from the exact rounding within
 * a few float32 spacings of x at a rounding boundary of the E4M3 grid.
 */
size_t fp4attn_quantize_v_e4m3_workspace_bytes(int B, int H, int N, int d);
int fp4attn_quantize_v_e4m3(const void* x_bf16, int B, int H, int N, int d, void* bytes_out, float* unit_scale_out,
                            void* workspace, size_t workspace_bytes, fp4attn_stream_t stream);

/* Bytes of device scratch fp4attn_attention_host needs for a problem of this size. */
size_t fp4attn_attention_host_workspace_bytes(int qk_fmt, int B, int H, int N, int d);

/*
 * Whole path from HOST buffers: copies bf16 Q, K, V [B,H,N,d] from (preferably pinned) host
 * memory into the caller's device workspace, quantizes them (fp4attn_quantize x3), runs
 * fp4attn_fwd and copies O (bf16) and, if LSE_host is not NULL, LSE back to host memory; returns
 * after enqueuing.  q_host/k_host/v_host/O_host/LSE_host are HOST pointers, workspace is a DEVICE
 * pointer of at least fp4attn_attention_host_workspace_bytes() bytes, 256-byte aligned.  The caller
 * synchronises `stream` before reading O_host: everything the call enqueues has completed by then.
 *
 * With MXFP4 Q, K and at least 8 (batch, head) units the call is pipelined over groups of units (they
 * are independent and MXFP4 needs no tensor-wide pass): the copy in of one group, the kernels of the
 * previous one and the copy out of the one before overlap, so the path costs about its largest leg
 * instead of the sum.  The copies then run on two internal streams (created on the first such call per
 * device and kept until the process exits; no device memory is allocated) that fork from `stream` and
 * join back into it through events.  NVFP4 (tensor-wide amax first) and small problems run on `stream`
 * alone.  Results are bit-identical either way.
 *
 * status_host (HOST pointer, preferably pinned; may be NULL): the call keeps a status word in its workspace,
 * clears it before its first kernel, hands it to every attention launch and copies it to *status_host at the
 * end: FP4ATTN_OK, or FP4ATTN_ERR_TIMEOUT if a bounded in-kernel wait ran out (O_host is then unspecified).
 * Read it after synchronising `stream`.
 *
 * Threads: every entry point may be called from several host threads (each on its own stream and
 * buffers); the pipelined host path serialises its enqueue phase on an internal lock because the
 * copy streams and events are shared per device.  On an error return the call still joins the
 * internal streams into `stream`, so whatever was enqueued stays ordered before later work there.
 */
int fp4attn_attention_host(const void* q_host, const void* k_host, const void* v_host,
                           int qk_fmt, float softmax_scale, int B, int H, int N, int d,
                           void* O_host, float* LSE_host, int* status_host,
                           void* workspace, size_t workspace_bytes, fp4attn_stream_t stream);

/*
 * Gives back what the library keeps between calls: the copy streams and events of fp4attn_attention_host on
 * every device that used it (they are created again on the next such call) and all cached tensor maps.  No
 * call of this library may be running or enqueuing on another thread, and every stream handed to
 * fp4attn_attention_host must have been synchronised.  Optional: a process that never calls it leaks nothing
 * but those objects until it exits.  (The paper has no counterpart.)
 */
int fp4attn_release(void);

/*
 * Dense FP4 tensor-core ceiling of the current device, measured: every SM issues `iters`
 * back-to-back block-scaled 128x128x64 E2M1 products on shared-memory-resident tiles.
 * Enqueues one kernel; *cycles_out (device, 64-bit) receives the slowest SM's clock count.
 * Used by the benchmark to state the roofline denominator; not part of the attention path.
 */
int fp4attn_mma_peak_probe(int iters, unsigned long long* cycles_out, fp4attn_stream_t stream);

/*
 * Arithmetic ceiling of the softmax warps on the current device, measured: on every SM, sixteen warps (four per
 * scheduler, as in the attention kernel) each run the score -> code arithmetic of Algorithm "direct-p-pack" -
 * block maximum, block exponent (ceiling rule), the code map (`p_map` and `exact_pairs` as in
 * fp4attn_operands; other values: FP4ATTN_ERR_INVALID_ARG), E2M1 conversion and packing - on `iters`
 * (1 .. 2^20) blocks of 32 rows x 32 scores held in shared memory, with no tensor product, tensor-memory
 * access or hand-off around it.  Enqueues one kernel; cycles_out (device, TWO 64-bit words, the second is scratch)
 * receives in its first word the slowest warp's clock count, so that cycles / (4 * iters) is the clocks one
 * scheduler needs per block.  Used by the benchmark for the roofline of the softmax arithmetic; not part of the
 * attention path.
 */
int fp4attn_softmax_arith_probe(int p_map, int exact_pairs, int iters, unsigned long long* cycles_out,
                                fp4attn_stream_t stream);

/*
 * Self-test of the bounded in-kernel waits (the failure-detection path; the paper has no
 * counterpart).  Launches one warp that waits on a barrier nothing completes, with a limit of
 * `limit_cycles` SM clocks (1 .. 2^31), and writes to *device_status what the attention kernel
 * would: FP4ATTN_ERR_TIMEOUT once the limit has run out (expected), FP4ATTN_OK otherwise.  The warp
 * returns normally; the context stays usable.
 */
int fp4attn_selftest_bounded_wait(long long limit_cycles, int* device_status, fp4attn_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* FP4ATTN_H_ */
