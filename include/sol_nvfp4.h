/*
 * sol_nvfp4.h -- C ABI of the B200 (sm_100a) NVFP4 linear-layer library.
 *
 * The library computes the W4A4 linear layers of a diffusion-transformer rollout:
 *     Y = Q(X) . Q(W)^T + bias
 * where Q is the NVFP4 quantizer of the paper's Section 2 ("FP4 Quantization and
 * Hardware Acceleration"):  x~ = S * Pi_FP4(x / S), FP4 = E2M1 (1 sign, 2 exponent,
 * 1 mantissa bit), one E4M3 scale per 16 contiguous elements along K.  S is split in two
 * levels: the E4M3 block scale and one FP32 scale T per tensor.  A BF16 linear of the
 * same shape is the full-precision reference the paper's second stage runs in.
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless its comment says host.  The caller owns
 *     every buffer; the library allocates no device memory (it keeps a small host-side
 *     cache of TMA descriptors and reads device properties once).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     All work is asynchronous on it; no call synchronises or reads device scalars on the
 *     host.  T flows from kernel to kernel through device memory.
 *   - Every function returns a sol_status_t; nothing throws.  Arguments are validated on
 *     the host before anything is launched: on an error status no kernel was launched.
 *   - Matrices are row-major with the K dimension contiguous: X is [M, K], W is [N, K]
 *     (the nn.Linear convention), Y is [M, N].  ld* are row pitches in ELEMENTS.
 *   - Requirements: M, N, K > 0; K % 32 == 0; N % 8 == 0; pointers 16-byte aligned; BF16
 *     row pitches multiples of 8 elements.  Inputs must be finite.
 *   - Only sm_100 devices are supported (SOL_ERR_UNSUPPORTED_ARCH otherwise); there is
 *     no CPU path.
 *   - A launch the CUDA runtime rejects returns SOL_ERR_CUDA; with the environment variable
 *     SOL_NVFP4_VERBOSE set, the runtime's error string is also printed to stderr.
 *
 * NVFP4 storage
 *   data   : uint8 [rows, K/2]; byte j of a row holds element 2j in its low nibble and
 *            element 2j+1 in its high nibble; nibble = s e e m.
 *   scales : uint8 E4M3 (unsigned use).  SOL_SF_ROW_MAJOR: [rows, K/16].
 *            SOL_SF_SWIZZLED_128x4: 512-byte chunks of 128 rows x 4 blocks, chunk order
 *            [ceil(rows/128)][ceil(K/64)]; inside a chunk the scale of (row r, block b) is at
 *            (r%32)*16 + ((r%128)/32)*4 + b%4.  Padding bytes are written as 0.  This is
 *            the layout the tensor core's scale-factor copy consumes; the GEMM entries
 *            require it.
 *   T      : one float; dequantized value = E2M1(nibble) * E4M3(scale) * T.
 */
#ifndef SOL_NVFP4_H_
#define SOL_NVFP4_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SOL_OK = 0,
    SOL_ERR_NULL_POINTER = 1,
    SOL_ERR_BAD_SHAPE = 2,
    SOL_ERR_ALIGNMENT = 3,
    SOL_ERR_WORKSPACE_TOO_SMALL = 4,
    SOL_ERR_UNSUPPORTED_ARCH = 5,
    SOL_ERR_CUDA = 6,
    SOL_ERR_TIMEOUT = 7,
    SOL_ERR_BAD_LAYOUT = 8
} sol_status_t;

typedef enum { SOL_SF_ROW_MAJOR = 0, SOL_SF_SWIZZLED_128x4 = 1 } sol_sf_layout_t;
typedef enum { SOL_ACT_NONE = 0, SOL_ACT_GELU_TANH = 1 } sol_activation_t;

/* Static, human-readable name of a status (host pointer, never NULL). */
const char *sol_status_string(sol_status_t status);

/* Bytes of packed FP4 data for a [rows, K] tensor: rows * K / 2.  0 on bad arguments. */
size_t sol_nvfp4_data_bytes(int64_t rows, int64_t K);

/* Bytes of the scale buffer in the given layout (swizzled: ceil(rows/128) * ceil(K/64) * 512).
 * 0 on bad arguments. */
size_t sol_nvfp4_scale_bytes(int64_t rows, int64_t K, sol_sf_layout_t layout);

/* Bytes of workspace nvfp4_quantize_linear needs for an [M, K] activation: packed data,
 * swizzled scales and one float, each region 256-byte aligned.  0 on bad arguments. */
size_t sol_nvfp4_linear_workspace_bytes(int64_t M, int64_t N, int64_t K);

/*
 * Per-tensor scale (second scaling level; the paper's single S is split so that block
 * scales span E4M3's range):  T = max|x| / (6 * 448), or 1 for an all-zero tensor.
 *   x                [rows, K] BF16, pitch ld
 *   tensor_scale_out one float (device), overwritten
 * The max is exact (order-independent), so the result is deterministic.
 */
sol_status_t sol_amax_bf16(const void *x, int64_t rows, int64_t K, int64_t ld,
                           float *tensor_scale_out, void *stream);

/*
 * Activation quantizer, Section 2's Q(x) with S = block scale * T.  Per row and per block
 * of 16 elements along K, in IEEE binary32 (round-to-nearest-even, no contraction):
 *     a = max|x|;  sb = E4M3_rne_sat(a / (6*T));  rcp = 1 / (float(sb) * T)  (0 if sb == 0)
 *     nibble_k = E2M1_rne_sat(x_k * rcp)   (ties to the even code, sign bit of x kept)
 *   x_bf16       [M, K] BF16, pitch ldx
 *   tensor_scale one float (device), read by the kernel; > 0
 *   q_out        sol_nvfp4_data_bytes(M, K) bytes
 *   sf_out       sol_nvfp4_scale_bytes(M, K, layout) bytes; every byte is written
 */
sol_status_t nvfp4_quantize(const void *x_bf16, int64_t M, int64_t K, int64_t ldx,
                            const float *tensor_scale, void *q_out, void *sf_out,
                            sol_sf_layout_t layout, void *stream);

/*
 * Weight quantizer: the same mapping applied to W [N, K] along K, preceded by the
 * per-tensor scale of W (the paper re-quantizes the policy weights after each update,
 * Section 3.4 / Appendix B.2).
 *   tensor_scale_out one float (device), written by the first kernel, read by the second
 */
sol_status_t nvfp4_quantize_weight(const void *w_bf16, int64_t N, int64_t K, int64_t ldw,
                                   void *q_out, void *sf_out, float *tensor_scale_out,
                                   sol_sf_layout_t layout, void *stream);

/*
 * Weight refresh: merge rank-r adapters into the base weights and quantize the result, the step
 * that follows every policy update (Section 3.4, Appendix B.2; Section 4.1: r = 32, alpha = 64,
 * so scaling = alpha / r = 2).  The paper does not spell the merge out; this is the usual
 *     W'[n][k] = bf16_rne( fma(scaling, acc, W[n][k]) ),
 *     acc = 0;  acc = fma(B[n][j], A[j][k], acc)  for j = 0 .. r-1 in this order   (IEEE binary32)
 * followed by nvfp4_quantize_weight's mapping applied to W'.
 *   w_bf16      [N, K] BF16, pitch ldw; not modified (training keeps base and adapters apart)
 *   lora_a      [r, K] BF16, pitch lda ("down" projection)
 *   lora_b      [N, r] BF16, pitch ldb ("up" projection); 1 <= r <= 64
 *   merged_bf16 [N, K] BF16, dense; receives W' (also the scratch the quantizer reads back)
 *   q_out, sf_out, layout: as for nvfp4_quantize_weight
 *   tensor_scale_out  TWO floats (device): [0] receives T of W'; [1] is scratch (it is left holding
 *                     max|W'|, the value T was derived from)
 * Three launches on the stream: clear the scratch word, the merge kernel, the quantizer.
 */
sol_status_t nvfp4_requantize_lora(const void *w_bf16, int64_t ldw, const void *lora_a, int64_t lda,
                                   const void *lora_b, int64_t ldb, int64_t N, int64_t K, int64_t r,
                                   float scaling, void *merged_bf16, void *q_out, void *sf_out,
                                   float *tensor_scale_out, sol_sf_layout_t layout, void *stream);

/*
 * The same for `count` matrices of one shape (all targeted projections of a model after a policy
 * update), in one call.  One matrix is ~20 us of GPU work, so launches are shared: matrices are
 * processed in groups of up to min(merged_matrices, 8), three launches per group.  The six lists
 * are HOST arrays of `count` DEVICE pointers; matrix i uses w_list[i] [N, K], a_list[i] [r, K],
 * b_list[i] [N, r] (all dense) and writes q_list[i], sf_list[i], ts_list[i] (two floats each).
 *   merged_bf16      device scratch for `merged_matrices` (>= 1) dense [N, K] BF16 matrices, reused
 *                    group after group in stream order (contents undefined afterwards); a scratch
 *                    that fits L2 keeps the merged weights out of HBM
 * Everything is validated before the first launch.
 */
sol_status_t nvfp4_requantize_lora_batch(int64_t count, const void *const *w_list, const void *const *a_list,
                                         const void *const *b_list, void *const *q_list, void *const *sf_list,
                                         float *const *ts_list, int64_t N, int64_t K, int64_t r, float scaling,
                                         void *merged_bf16, int64_t merged_matrices, sol_sf_layout_t layout,
                                         void *stream);

/*
 * Block-scaled FP4 GEMM with BF16 output (the NVFP4 linear the rollout runs, Section 3.4):
 *     acc[m,n] = sum_b sx[m,b] * sw[n,b] * sum_{k in b} qx[m,k] * qw[n,k]      (FP32 accumulate)
 *     Y[m,n]   = bf16_rne( fma(acc, Tx*Tw, bias[n]) )
 *   xq, wq     packed data [M, K/2], [N, K/2] (dense pitch K/2 bytes)
 *   xsf, wsf   scales in SOL_SF_SWIZZLED_128x4 layout
 *   x_tscale, w_tscale   one float each (device)
 *   bias_bf16  [N] BF16 or NULL
 *   y_bf16     [M, N] BF16, pitch ldy
 */
sol_status_t nvfp4_linear(const void *xq, const void *xsf, const float *x_tscale,
                          const void *wq, const void *wsf, const float *w_tscale,
                          const void *bias_bf16, void *y_bf16, int64_t M, int64_t N, int64_t K,
                          int64_t ldy, void *stream);

/*
 * The NVFP4 linear with its output already quantized for the NEXT NVFP4 linear: between two
 * rollout linears (Section 3.4) the activations never exist in BF16 in memory, which removes the
 * 2 B/element store, the amax pass and the 2.56 B/element quantizer pass of the next layer.
 *     y[m,n] = fma(acc[m,n], Tx*Tw, bias[n])                     (as nvfp4_linear, FP32)
 *     h[m,n] = bf16_rne( act(y[m,n]) )       act = identity or GELU (tanh form), FP32
 *     (hq, hsf) = the activation quantizer of nvfp4_quantize applied to h along N with T = *out_tscale
 * The two-level scale needs T before the first output exists, so T is the caller's: a calibrated
 * value or the one derived from the previous step's amax_out (a value too small only saturates
 * more blocks at 6*448*T).
 *   out_tscale  one float (device), > 0
 *   hq_out      packed nibbles [M, N/2];  hsf_out  scales, SOL_SF_SWIZZLED_128x4 layout of an [M, N]
 *               tensor, sol_nvfp4_scale_bytes(M, N, ...) bytes, padding rows written as 0
 *   amax_out    nullable; one device word holding max|h| as an FP32 value, updated with an atomic
 *               max (a running maximum: the caller zeroes it to start a new window)
 *   N % 64 == 0.  GELU is evaluated in FP32 with the hardware tanh (absolute error of tanh about
 *   2^-11): far below the BF16 rounding and the FP4 grid that follow, but h can differ from an exactly
 *   evaluated GELU in its last BF16 place more often than the GEMM's accumulation order alone causes.
 */
sol_status_t nvfp4_linear_quantized_out(const void *xq, const void *xsf, const float *x_tscale, const void *wq,
                                        const void *wsf, const float *w_tscale, const void *bias_bf16,
                                        sol_activation_t activation, const float *out_tscale, void *hq_out,
                                        void *hsf_out, float *amax_out, int64_t M, int64_t N, int64_t K,
                                        void *stream);

/*
 * The same for a linear whose outputs feed two consumers, as the first linear of a single-stream
 * DiT block does (3072 -> 9216 + 12288 in the FLUX-shaped config): columns [0, n_split) leave as BF16
 * (q, k, v for attention); columns [n_split, N) pass through the activation and leave quantized
 * into columns [dest_col0, dest_col0 + N - n_split) of a WIDER quantized tensor [M, dest_K] -- the
 * concatenated input of the next linear, whose other columns nvfp4_quantize_into fills.
 *   y_bf16      [M, n_split] BF16, pitch ldy
 *   hq_dest     packed nibbles [M, dest_K/2];  hsf_dest  chunked scales of an [M, dest_K] tensor
 *   out_tscale  the tensor scale of the whole destination tensor (one T for all its parts)
 *   n_split % 256 == 0, (N - n_split) % 64 == 0, dest_K % 64 == 0, dest_col0 % 64 == 0.
 * Everything else as nvfp4_linear_quantized_out.
 */
sol_status_t nvfp4_linear_split_out(const void *xq, const void *xsf, const float *x_tscale, const void *wq,
                                    const void *wsf, const float *w_tscale, const void *bias_bf16, void *y_bf16,
                                    int64_t ldy, int64_t n_split, sol_activation_t activation,
                                    const float *out_tscale, void *hq_dest, void *hsf_dest, int64_t dest_K,
                                    int64_t dest_col0, float *amax_out, int64_t M, int64_t N, int64_t K,
                                    void *stream);

/*
 * nvfp4_quantize writing into columns [dest_col0, dest_col0 + K) of a wider quantized tensor
 * [M, dest_K] (chunked scale layout): the part of a concatenated activation that arrives in BF16.
 * K, dest_K and dest_col0 are multiples of 64; bytes outside the column range are not touched, so
 * the rows past M of the destination's last 128-row scale chunk must have been zeroed once.
 */
sol_status_t nvfp4_quantize_into(const void *x_bf16, int64_t M, int64_t K, int64_t ldx, const float *tensor_scale,
                                 void *q_dest, void *sf_dest, int64_t dest_K, int64_t dest_col0, void *stream);

/*
 * The quantizer fused into the other producer of a DiT linear's input: an adaptive layer norm.
 *     mu, var = mean and population variance of row m;  xhat = (x - mu) / sqrt(var + eps)   (FP32)
 *     h[m,k]  = bf16_rne( xhat[k] * (1 + scale[s,k]) + shift[s,k] ),   s = m / rows_per_sample
 *     (q, sf) = nvfp4_quantize's mapping applied to h with T = *tensor_scale (caller supplied)
 * One pass over x: 2 B read and 0.56 B written per element instead of a norm pass, an amax pass
 * and a quantizer pass.
 *   x_bf16       [M, K] BF16, pitch ldx;  K % 64 == 0, K <= 4096
 *   scale, shift [ceil(M / rows_per_sample), K] BF16, dense (the per-sample modulation)
 *   q_out        [M, K/2];  sf_out  SOL_SF_SWIZZLED_128x4 scales of an [M, K] tensor, every byte written
 *   amax_out     nullable running max|h| (atomic max on the FP32 value), as in nvfp4_linear_quantized_out
 */
sol_status_t nvfp4_layernorm_quantize(const void *x_bf16, int64_t M, int64_t K, int64_t ldx, const void *scale_bf16,
                                      const void *shift_bf16, int64_t rows_per_sample, float eps,
                                      const float *tensor_scale, void *q_out, void *sf_out, float *amax_out,
                                      void *stream);

/*
 * Scaled-dot-product attention of a DiT block in BF16 (the rollout models of Section 4.1 are
 * diffusion transformers; the method quantizes their linear layers, Section 3, and leaves attention
 * in BF16 in the FP4 and in the BF16 path alike):
 *     out[b, s, h, :] = sum_t softmax_t( q[b,s,h,:] . k[b,t,h,:] / sqrt(head_dim) ) v[b,t,h,:]
 * No mask, no dropout; head_dim is 128 (FLUX.1) or 64 (SD3.5).  Scores and sums in FP32, probabilities rounded to BF16
 * before the product with V, output rounded to BF16.
 *   q, out   [batch, seq_q, heads, head_dim] BF16: element (b, s, h, d) at ((b * seq_q + s) * ld + h * head_dim + d),
 *            ld_q / ld_out elements between consecutive tokens (>= heads * head_dim, multiple of 8), so q, k
 *            and v may be column slices of one fused projection output
 *   k, v     [batch, seq_kv, heads, head_dim] BF16, the same way with ld_k / ld_v
 * All pointers are device pointers, 16-byte aligned, owned by the caller; out must not alias an input.
 * Errors: SOL_ERR_NULL_POINTER, SOL_ERR_BAD_SHAPE (a non-positive extent, another head_dim, ld < heads * head_dim,
 * heads or batch above 65535), SOL_ERR_ALIGNMENT, SOL_ERR_UNSUPPORTED_ARCH, SOL_ERR_CUDA; nothing is launched on an error.
 */
sol_status_t sol_attention_bf16(const void *q, const void *k, const void *v, void *out, int64_t batch, int64_t seq_q,
                                int64_t seq_kv, int64_t heads, int64_t head_dim, int64_t ld_q, int64_t ld_k, int64_t ld_v,
                                int64_t ld_out, void *stream);

/*
 * sol_attention_bf16 whose output leaves as the quantized activations of the linear that follows it in
 * a DiT block (the output projection; in a single-stream block the concatenated input it shares
 * with the MLP branch): h = bf16(attention output), then nvfp4_quantize's mapping with
 * T = *out_tscale, written into columns [dest_col0, dest_col0 + heads * head_dim) of the NVFP4 tensor
 * [batch * seq_q, dest_K] (rows of all samples stacked; chunked scale layout).  Bit for bit what
 * sol_attention_bf16 followed by nvfp4_quantize_into produces, without the BF16 round trip through HBM.
 *   out_tscale   caller supplied (a delayed scale); amax_out: nullable running max|h| as in
 *                nvfp4_linear_quantized_out
 *   dest_K % 64 == 0, dest_col0 % 64 == 0, dest_col0 + heads * head_dim <= dest_K
 * Bytes outside the column range are not touched, so the rows past batch * seq_q of the destination's
 * last 128-row scale chunk must have been zeroed once.  Everything else as sol_attention_bf16.
 */
sol_status_t sol_attention_nvfp4_out(const void *q, const void *k, const void *v, int64_t batch, int64_t seq_q,
                                     int64_t seq_kv, int64_t heads, int64_t head_dim, int64_t ld_q, int64_t ld_k, int64_t ld_v,
                                     const float *out_tscale, void *q_dest, void *sf_dest, int64_t dest_K,
                                     int64_t dest_col0, float *amax_out, void *stream);

/*
 * The same attention over two token streams that are projected separately and attend jointly, as in
 * the double-stream blocks of the FLUX.1 model of Section 4.1 (text tokens and image tokens): the
 * joint sequence is the first stream's tokens followed by the second's; queries, keys and values
 * are read from, and outputs written to, each stream's own tensors -- no concatenated copy exists.
 *   first, second   host pointers to the two descriptions below (read during the call only);
 *                   q, k, v, out: device pointers laid out as in sol_attention_bf16, `seq` tokens each
 *   first->seq % 256 == 0 (the first stream fills whole query-tile pairs); second->seq is free
 * Errors as for sol_attention_bf16, plus SOL_ERR_BAD_SHAPE for a first stream that is not a multiple
 * of 256 tokens.
 */
typedef struct {
    const void *q, *k, *v;
    void *out;
    int64_t seq, ld_q, ld_k, ld_v, ld_out;
} sol_attention_stream_t;
sol_status_t sol_attention_bf16_joint(const sol_attention_stream_t *first, const sol_attention_stream_t *second,
                                      int64_t batch, int64_t heads, int64_t head_dim, void *stream);

/*
 * BF16 linear, the full-precision stage-2 reference (Section 3.4):
 *     Y[m,n] = bf16_rne( sum_k x[m,k] * w[n,k] + bias[n] ),  FP32 accumulate.
 */
sol_status_t bf16_linear(const void *x_bf16, const void *w_bf16, const void *bias_bf16,
                         void *y_bf16, int64_t M, int64_t N, int64_t K, int64_t ldx,
                         int64_t ldw, int64_t ldy, void *stream);

/*
 * Fused entry: dynamic per-tensor scale of X, quantize X, NVFP4 GEMM against
 * pre-quantized weights, in one call on one stream.
 *   workspace  device scratch of at least sol_nvfp4_linear_workspace_bytes(M, N, K) bytes,
 *              256-byte aligned; holds Q(X) between the kernels; contents undefined after.
 */
sol_status_t nvfp4_quantize_linear(const void *x_bf16, int64_t ldx, const void *wq,
                                   const void *wsf, const float *w_tscale,
                                   const void *bias_bf16, void *y_bf16, int64_t M, int64_t N,
                                   int64_t K, int64_t ldy, void *workspace,
                                   size_t workspace_bytes, void *stream);

/*
 * The fused entry without the amax pass ("delayed" tensor scale): X is quantized with the T the
 * caller carries over from an earlier call on the same activation stream, and the amax of THIS X
 * is collected by the quantizer as a by-product (it computes every block maximum anyway), so the
 * second HBM read of X disappears.  A T that has become too small only saturates more block scales.
 *   scale_state  two floats (device, 8-byte aligned): [0] = T used by this call (> 0; read only),
 *                [1] = running max|x| as an FP32 value, raised by this call with an atomic max
 *   sol_roll_tensor_scale(state): [0] <- max|x| / 2688 (1 if it is 0), [1] <- 0 -- one tiny kernel,
 *                called between denoising steps (or whenever the caller wants T refreshed)
 * Given the same T the result is bit-identical to nvfp4_quantize + nvfp4_linear.
 */
sol_status_t nvfp4_quantize_linear_delayed(const void *x_bf16, int64_t ldx, const void *wq, const void *wsf,
                                           const float *w_tscale, const void *bias_bf16, void *y_bf16, int64_t M,
                                           int64_t N, int64_t K, int64_t ldy, float *scale_state, void *workspace,
                                           size_t workspace_bytes, void *stream);
sol_status_t sol_roll_tensor_scale(float *scale_state, void *stream);

/*
 * The fused entry for HOST activations and outputs (the end-to-end path a caller with data in host
 * memory takes): copies X host -> x_dev, runs nvfp4_quantize_linear, copies y_dev -> Y host, all
 * queued on `stream` (truly asynchronous only if the host buffers are pinned).
 *   x_host, y_host  HOST pointers, BF16 [M, K] / [M, N], pitches ldx / ldy in elements
 *   x_dev, y_dev    device staging buffers, dense [M, K] / [M, N] BF16, 16-byte aligned
 *   weights, bias, workspace: device, as for nvfp4_quantize_linear
 */
sol_status_t nvfp4_quantize_linear_host(const void *x_host, int64_t ldx, const void *wq,
                                        const void *wsf, const float *w_tscale,
                                        const void *bias_bf16, void *y_host, int64_t M, int64_t N,
                                        int64_t K, int64_t ldy, void *x_dev, void *y_dev,
                                        void *workspace, size_t workspace_bytes, void *stream);

/*
 * MXFP4, the OCP format Section 2 sets beside NVFP4: 32 contiguous elements along K under one E8M0
 * scale (a bare exponent: byte b = 2^(b-127)), no tensor-level scale.
 *     scale = 2^(floor(log2 max|x|) - 2), exponent clamped to [-127, 127]; byte 0 for an all-zero block
 *     nibble_k = E2M1_rne_sat(x_k / scale)    (the division is an exact power-of-two scaling)
 * Storage: nibbles as for NVFP4; scales row-major [rows, K/32], or SOL_SF_SWIZZLED_128x4: the same
 * 512-byte chunks of 128 rows x 4 scales (a chunk now spans 128 elements of K), chunk order
 * [ceil(rows/128)][ceil(K/128)], padding 0.  sol_mxfp4_scale_bytes gives the buffer size.
 */
size_t sol_mxfp4_scale_bytes(int64_t rows, int64_t K, sol_sf_layout_t layout);
sol_status_t mxfp4_quantize(const void *x_bf16, int64_t rows, int64_t K, int64_t ldx, void *q_out, void *sf_out,
                            sol_sf_layout_t layout, void *stream);

/*
 * MXFP4 linear: Y[m,n] = bf16_rne( sum_b 2^(ex[m,b] + ew[n,b]) sum_{k in b} qx[m,k] qw[n,k] + bias[n] ),
 * FP32 accumulation in the tensor core (kind::mxf4, two scales per row per K = 64 instruction).
 * Operands as written by mxfp4_quantize with the chunked scale layout; otherwise as nvfp4_linear.
 */
sol_status_t mxfp4_linear(const void *xq, const void *xsf, const void *wq, const void *wsf, const void *bias_bf16,
                          void *y_bf16, int64_t M, int64_t N, int64_t K, int64_t ldy, void *stream);

/*
 * mxfp4_linear whose output leaves as the MXFP4 activations of the next linear (the MXFP4 form of
 * nvfp4_linear_quantized_out): h = bf16_rne(act(Y)), then mxfp4_quantize's mapping along N.
 *   hq_out   [M, N/2] nibbles;  hsf_out  SOL_SF_SWIZZLED_128x4 MXFP4 scales of an [M, N] tensor, every byte written
 *   amax_out nullable running max|h| (FP32 bits, atomic max); N % 128 == 0
 * No tensor scales anywhere: the format has none.  Errors as nvfp4_linear_quantized_out.
 */
sol_status_t mxfp4_linear_quantized_out(const void *xq, const void *xsf, const void *wq, const void *wsf,
                                        const void *bias_bf16, sol_activation_t activation, void *hq_out, void *hsf_out,
                                        float *amax_out, int64_t M, int64_t N, int64_t K, void *stream);

/*
 * The MXFP4 forms of nvfp4_linear_split_out and nvfp4_quantize_into (Section 2 names MXFP4 beside NVFP4;
 * the concatenated input of a single-stream block's second linear, as there): columns [0, n_split) of the
 * linear leave as BF16, columns [n_split, N) pass through the activation and leave as MXFP4 into columns
 * [dest_col0, dest_col0 + N - n_split) of a wider MXFP4 tensor [M, dest_K]; mxfp4_quantize_into quantizes a
 * BF16 tensor [M, K] into columns [dest_col0, dest_col0 + K) of such a tensor and touches no other column.
 *   hq_dest / q_dest  packed nibbles [M, dest_K/2];  hsf_dest / sf_dest  chunked MXFP4 scales of an [M, dest_K] tensor
 *   n_split % 256 == 0;  N - n_split, K, dest_K and dest_col0 multiples of 128 (a scale chunk spans 128 columns).
 * No tensor scale: the format has none.  Errors as the NVFP4 forms.
 */
sol_status_t mxfp4_linear_split_out(const void *xq, const void *xsf, const void *wq, const void *wsf,
                                    const void *bias_bf16, void *y_bf16, int64_t ldy, int64_t n_split,
                                    sol_activation_t activation, void *hq_dest, void *hsf_dest, int64_t dest_K,
                                    int64_t dest_col0, float *amax_out, int64_t M, int64_t N, int64_t K, void *stream);
sol_status_t mxfp4_quantize_into(const void *x_bf16, int64_t M, int64_t K, int64_t ldx, void *q_dest, void *sf_dest,
                                 int64_t dest_K, int64_t dest_col0, void *stream);

/*
 * Stage-1 selection (Section 3.4; Section 4.1 "Rollout Generation": N = 96 candidates per prompt,
 * the 12 best and 12 worst kept, their initial noises preserved) and the group-standardised
 * advantages of the GRPO equation in Section 2, A_i = (R_i - mean) / population std.
 *   rewards        [P, N] FP32 proxy rewards, finite; N <= 4096
 *   seeds          [P, N] 64-bit noise seeds (nullable when seeds_out is null)
 *   idx_out        [P, K] int32: K/2 best candidates in descending order of reward, then the K/2
 *                  worst starting from the lowest; among equal rewards the lower index ranks higher
 *   seeds_out      [P, K] the selected candidates' seeds (nullable)
 *   advantages_out [P, N] FP32 (nullable); statistics in FP64; all zeros when the std is 0
 *   K even, 0 < K <= N.  One block per prompt; indices and seeds are exact.
 */
sol_status_t solrl_select_contrastive(const float *rewards, const uint64_t *seeds, int64_t P, int64_t N, int64_t K,
                                      int32_t *idx_out, uint64_t *seeds_out, float *advantages_out, void *stream);

/*
 * Rank consistency between reference and proxy rewards (appendix "Group-Relative Ranking
 * Consistency"): per prompt
 *   counts_out  [P, 4] int64: concordant minus discordant pairs (ties count 0), sum of squared
 *               rank differences (ordinal ranks, ties to the lower index), candidates in both top-k
 *               sets, candidates in both bottom-k sets -- all exact
 *   metrics_out [P, 4] FP32 (nullable): Kendall tau-a = count / (N(N-1)/2), Spearman rho =
 *               1 - 6 sum d^2 / (N(N^2-1)), top-k and bottom-k match rates
 *   2 <= N <= 2048, 0 < k <= N.
 */
sol_status_t solrl_rank_consistency(const float *rewards_ref, const float *rewards_proxy, int64_t P, int64_t N,
                                    int64_t k, int64_t *counts_out, float *metrics_out, void *stream);

/*
 * (No counterpart in the paper: an addition for callers that cannot allocate device memory.)
 *
 * Same computation and result as nvfp4_quantize_linear, but without a workspace argument: the
 * scratch for the quantized activations lives in a fixed 64 MiB device array that is part of the
 * library image, so the call performs no device allocation of any kind.  It is meant for callers
 * that are handed input and output buffers only, or that run after their memory pool has been
 * frozen (serving loops, plugins, frameworks that forbid allocation once set up).
 *   - Problems whose scratch (sol_nvfp4_linear_workspace_bytes(M, N, K)) exceeds
 *     sol_nvfp4_static_scratch_bytes() are rejected with SOL_ERR_WORKSPACE_TOO_SMALL; nothing is launched.
 *   - The first call on each device looks up the array's device address (with that device current);
 *     make that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents.  Calls
 *     that may overlap on the GPU (different streams, or several host threads) race on it and give
 *     undefined results; serialise them.  Every GPU that loads the library holds the array until
 *     the process exits.
 */
size_t sol_nvfp4_static_scratch_bytes(void);
sol_status_t nvfp4_quantize_linear_static(const void *x_bf16, int64_t ldx, const void *wq,
                                          const void *wsf, const float *w_tscale,
                                          const void *bias_bf16, void *y_bf16, int64_t M, int64_t N,
                                          int64_t K, int64_t ldy, void *stream);

/*
 * Device-side waits in the GEMM kernels are bounded; a wait that runs out records a code
 * in a device status word and the kernel returns.  This call synchronises `stream`, reads
 * that word, clears it, and returns SOL_ERR_TIMEOUT if it was set, SOL_ERR_CUDA if the
 * stream reported an error, SOL_OK otherwise.  `detail_out` (host, nullable) receives the
 * raw word.
 */
sol_status_t sol_last_device_status(void *stream, uint32_t *detail_out);

/*
 * (No counterpart in the paper: failure detection of the kernels themselves.)
 *
 * Sets, for the current device, the limit of every bounded device-side wait in SM clock cycles
 * (default 4e9, about two seconds; `cycles` <= 0 restores the default).  Synchronous: it copies
 * eight bytes to the device and affects kernels launched afterwards.  A wait that exceeds the limit
 * makes its kernel leave through the normal teardown (outputs incomplete) and is reported by
 * sol_last_device_status as SOL_ERR_TIMEOUT; the context stays usable.
 */
sol_status_t sol_set_wait_limit_cycles(int64_t cycles);

/*
 * Test hook for that path (no counterpart in the paper).  While `on` is non-zero on the current
 * device, the load-issuing warps of the CTA-pair GEMM kernels (M > 128: nvfp4_linear, mxfp4_linear,
 * bf16_linear and the entries built on them) issue no loads, so every consumer wait of such a launch
 * runs into the wait limit: nothing traps, faults or spins without bound, the kernel returns with Y
 * unwritten and the status word set.  Use it with a short limit (about 1e6 cycles) and switch it off
 * again; it is not meant for anything but exercising the time-out path.
 */
sol_status_t sol_test_hold_loads(int on);

#ifdef __cplusplus
}
#endif
#endif /* SOL_NVFP4_H_ */
