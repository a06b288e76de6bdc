/*
 * ibert.h -- C ABI of the B200 (sm_100a) integer-only Transformer encoder layer
 * of I-BERT (Kim et al., "I-BERT: Integer-only BERT Quantization").
 *
 * Every call takes quantized tensors in the paper's (q, S) convention
 * (Sec. 3.1: real value = S * q, S fixed offline) and returns (q', S').
 * Kernels never see a scale: the host turns scales into integer constants
 * before the launch (static quantization; footnote of Algorithm 1).
 *
 * General rules
 *   - Tensor pointers are DEVICE pointers owned by the caller, 16-byte
 *     aligned, row-major and contiguous unless stated otherwise.
 *     Scale arrays, gamma/beta and everything inside ibert_layer_desc are
 *     HOST pointers, read during the call and not retained.
 *   - Work is enqueued on the stream given to ibert_create(); calls return
 *     without synchronizing (ibert_last_status() synchronizes).
 *   - Every function returns IBERT_OK (0) or a negative IBERT_ERR_* code;
 *     nothing throws (a failed host allocation is IBERT_ERR_NOMEM), aborts,
 *     or falls back to a CPU path.  Invalid
 *     arguments are rejected on the host before anything is launched.
 *   - Device-side waits are bounded (one second on the GPU's timer); if one
 *     expires the kernel records IBERT_ERR_TIMEOUT in the context's status
 *     word and returns normally.
 *   - Value formats: "int8" = [-127,127] in int8_t; "Q16" = [-32767,32767]
 *     in an int32_t container; "u8" = [0,255] in uint8_t.
 *   - Requantization (Appendix C.1, dyadic form b / 2^c):
 *       requant(v; b, c, qmax) = clamp((v*b + (c>0 ? 2^(c-1) : 0)) >> c, +-qmax)
 *     with the product in 64 bits, >> arithmetic, 0 <= c <= 31, |b| < 2^31.
 */
#ifndef IBERT_H_
#define IBERT_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define IBERT_OK 0
#define IBERT_ERR_ARG (-1)         /* null pointer, bad enum, negative size      */
#define IBERT_ERR_SHAPE (-2)       /* size outside the supported range           */
#define IBERT_ERR_SCALE_RANGE (-3) /* scale not finite/positive or not dyadic-representable */
#define IBERT_ERR_ALIGN (-4)       /* pointer or row pitch not 16-byte aligned   */
#define IBERT_ERR_NOMEM (-5)       /* device or host allocation failed           */
#define IBERT_ERR_CUDA (-6)        /* a CUDA runtime / driver call failed        */
#define IBERT_ERR_TIMEOUT (-7)     /* a bounded device-side wait expired         */
#define IBERT_ERR_VALUE_RANGE (-8) /* an integer left the range the method assumes */

typedef struct ibert_ctx ibert_ctx;     /* device, stream, workspace, status word        */
typedef struct ibert_layer ibert_layer; /* one layer's device-resident integer parameters */

/* Creates a context on `device` that launches on `cuda_stream` (a cudaStream_t; NULL =
   the legacy default stream).  The context owns a small device status word and caches of
   derived constant tables. */
int ibert_create(ibert_ctx** out, int device, void* cuda_stream);
int ibert_destroy(ibert_ctx* ctx);
/* Synchronizes the context's stream and returns the first device-side error recorded since
   the last call (IBERT_OK if none), or IBERT_ERR_CUDA if the stream is in error. */
int ibert_last_status(ibert_ctx* ctx);
const char* ibert_strerror(int code);

/* Host, pure.  Real multiplier m -> (b, c) with m ~= b / 2^c (Appendix C.1; the dyadic
   form of the cited requantization scheme): c = min(31, 31 - exponent(m)),
   b = round-half-up(|m| * 2^c) with the sign of m, renormalized if it reaches 2^31.
   IBERT_ERR_SCALE_RANGE if |m| >= 2^31 or m is not finite. */
int ibert_dyadic_from_double(double m, int32_t* b, int32_t* c);

/* INT8 MatMul with INT32 accumulation (Sec. 2, Appendix C.1), bias add and requantization:
     acc[m,n] = sum_k x[m,k] * w[n,k] + bias[n];   out = requant(acc; dyadic(S_x*S_w[n]/S_out))
   x [M,K] int8, w [N,K] int8 (K contiguous), bias [N] int32 at scale S_x*S_w[n] (may be NULL),
   S_w host array [N] (per-output-channel weight scales).
   out_kind 0: out is int8 [M,N] at S_out;  1: out is Q16 in int32 [M,N] at S_out;
            2: out is the raw int32 accumulators (S_out ignored);
            3: out is Q16 in int16 [M,N] at S_out -- the values of kind 1 in half the bytes (the
               "INT32 precision" inputs of the non-linear operations, Sec. 3.6 / Appendix C.1, are
               brought to a per-tensor scale and then never exceed 16 bits).
   S_ret (host, may be NULL): receives S_out (kinds 0, 1, 3: one entry) or S_x*S_w[n] (kind 2: N entries).
   Requires K % 16 == 0, N % 16 == 0 (kind 0) / N % 4 == 0 (kinds 1, 2) / N % 8 == 0 (kind 3),
   K*127*127 + |bias| < 2^31, M < 2^31 - 256. */
int ibert_linear_i8(ibert_ctx* ctx, const int8_t* x, double S_x, const int8_t* w, const double* S_w,
                    const int32_t* bias, int64_t M, int N, int K, int out_kind, double S_out,
                    void* out, double* S_ret);

/* Same product followed by i-GELU (Algorithm 2) in the epilogue -- the FFN1 step:
   acc -> Q16 at S_mid -> i-GELU -> int8 at S_out.  out is int8 [M,N]. */
int ibert_linear_gelu_i8(ibert_ctx* ctx, const int8_t* x, double S_x, const int8_t* w, const double* S_w,
                         const int32_t* bias, int64_t M, int N, int K, double S_mid, double S_out,
                         int8_t* out, double* S_ret);

/* i-softmax (Algorithm 3, Eq. 11-15) over rows of length L of int32 scores q at scale S:
   row max, i-exp (shift decomposition + 2nd-order polynomial), int32 row sum, fixed-point
   quotient p = floor(e * p_max / sum).  out is u8 [rows, L]; *S_ret = 1/p_max.
   L in [1,1024]; p_max in {255,127}; S <= ln 2 (else IBERT_ERR_SCALE_RANGE). */
int ibert_softmax_i(ibert_ctx* ctx, const int32_t* q, double S, int64_t rows, int L, int p_max,
                    uint8_t* out, double* S_ret);

/* i-softmax with i-exp by table look-up -- the alternative the paper argues against (Sec. 2,
   Sec. 3.5), here only for a measured comparison.  The table holds the i-exp of every pre-shifted
   distance from the row maximum, 0 .. 31*q_ln2 (up to 2 MiB of uint32), filled on first use for a
   scale by the same device function ibert_softmax_i evaluates, and cached in the context (at most 64
   tables, dropped together after a stream synchronization when a 65th is needed; freed by
   ibert_destroy).  Results are identical to ibert_softmax_i; arguments and errors as there, plus
   IBERT_ERR_NOMEM when the table cannot be allocated. */
int ibert_softmax_lut_i(ibert_ctx* ctx, const int32_t* q, double S, int64_t rows, int L, int p_max,
                        uint8_t* out, double* S_ret);

/* i-GELU (Algorithm 2, Eq. 8-9), elementwise.  q int32 at scale S, clamped to Q16 first;
   out int8 at S_out (the product q*(q_erf+q_1) is requantized in-kernel); *S_ret = S_out. */
int ibert_gelu_i(ibert_ctx* ctx, const int32_t* q, double S, int64_t n, double S_out, int8_t* out,
                 double* S_ret);

/* Residual add + i-LayerNorm (Sec. 3.6, Eq. 16, Algorithm 4) over rows of C channels:
     v = q + requant(r; dyadic(S_r/S)) (r may be NULL), mu = floor(sum v / C),
     sigma = max(ISqrt(floor(sum (v-mu)^2 / C)), 1), normalized, scaled by gamma, shifted by beta,
     requantized to int8 at S_out.
   q int32 [rows,C] at S (Q16-range values; |v| <= 2^20 is a documented, unchecked precondition),
   r int8 [rows,C] at S_r, gamma/beta host double[C].  C in [1,2047].  *S_ret = S_out. */
int ibert_layernorm_i(ibert_ctx* ctx, const int32_t* q, double S, const int8_t* r, double S_r,
                      const double* gamma, const double* beta, int64_t rows, int C, double S_out,
                      int8_t* out, double* S_ret);

/* The same operation on Q16 values stored as int16 (Sec. 3.6 / Appendix C.1: the LayerNorm input
   is the requantized accumulator of the preceding MatMul, at a per-tensor scale; in Q16 it fits 16
   bits): q int16 [rows,C], everything else, and every result, as ibert_layernorm_i on the same
   values.  4 instead of 6 bytes of traffic per element. */
int ibert_layernorm_i16(ibert_ctx* ctx, const int16_t* q, double S, const int8_t* r, double S_r,
                        const double* gamma, const double* beta, int64_t rows, int C, double S_out,
                        int8_t* out, double* S_ret);

/* The same operation for callers that cannot allocate device memory (no counterpart in the
   paper: a deployment convenience).  ibert_layernorm_i keeps its per-channel constant tables in
   memory it obtains with cudaMalloc; code that runs where allocation is forbidden -- inside a
   region that must not touch the allocator, under a memory budget owned by another component,
   or in a host thread that may not block on the driver's allocation lock -- can call this
   variant instead.  It needs no ibert_ctx: work is enqueued on `cuda_stream` (a cudaStream_t,
   NULL = legacy default stream) of the CURRENT device, and the tables plus a status word live in
   a fixed device array of 24,832 bytes that every GPU loading the library holds until exit.
   It calls no cudaMalloc / cudaFree nor any other routine that allocates device memory.
   Limits and caveats: C <= IBERT_STATIC_LN_MAX_C (larger C -> IBERT_ERR_SHAPE); all calls on a
   device share the one array, so two calls whose GPU work may overlap (different streams without
   ordering) race on it -- serialize them; the first call on each device looks up the array's
   device address, so make that first call outside any stream capture.
   Arguments and results are exactly those of ibert_layernorm_i.  A bounded wait that runs out
   inside the kernel is recorded in a status word inside the same array;
   ibert_layernorm_i_static_status synchronizes `cuda_stream`, returns that word for the current
   device (IBERT_OK or IBERT_ERR_TIMEOUT) and clears it; it allocates nothing either. */
#define IBERT_STATIC_LN_MAX_C 2047
int ibert_layernorm_i_static(void* cuda_stream, const int32_t* q, double S, const int8_t* r, double S_r,
                             const double* gamma, const double* beta, int64_t rows, int C, double S_out,
                             int8_t* out, double* S_ret);
int ibert_layernorm_i_static_status(void* cuda_stream);

/* Multi-head self-attention on int8 Q|K|V (Fig. 1 right: MatMul -> i-softmax -> MatMul):
   per (batch, head): s = Q K^T (int32, scale S_q*S_k/8, head size 64), p = i-softmax(s) in u8
   (p_max = 255) or 7-bit (p_max = 127), ctx = requant(p V; dyadic((1/p_max)*S_v/S_ctx)).
   qkv int8 [B*L, 3H] with column blocks Q | K | V, head j at columns 64j..64j+63 of each block;
   ctx int8 [B*L, H].  Scores never leave the SM.  L in [1,512], H = 64*heads. */
int ibert_attention_i8(ibert_ctx* ctx, const int8_t* qkv, int B, int L, int H, int heads, double S_q,
                       double S_k, double S_v, double S_ctx, int p_max, int8_t* out, double* S_ret);

/* One encoder layer's parameters; every pointer is a HOST pointer (copied at create). */
typedef struct ibert_layer_desc {
  int32_t H, heads, F, p_max;                 /* H = 64*heads; p_max in {255,127} */
  const int8_t* w_qkv; const double* S_w_qkv; const int32_t* bias_qkv; /* [3H,H], [3H], [3H] */
  const int8_t* w_o;   const double* S_w_o;   const int32_t* bias_o;   /* [H,H],  [H],  [H]  */
  const int8_t* w_f1;  const double* S_w_f1;  const int32_t* bias_f1;  /* [F,H],  [F],  [F]  */
  const int8_t* w_f2;  const double* S_w_f2;  const int32_t* bias_f2;  /* [H,F],  [H],  [H]  */
  const double* gamma1; const double* beta1;  /* [H] LayerNorm after attention */
  const double* gamma2; const double* beta2;  /* [H] LayerNorm after the FFN   */
  /* static activation scales: layer input, Q, K, V, context, first residual sum (Q16),
     LayerNorm-1 output, GELU input (Q16), GELU output, second residual sum (Q16), output */
  double S_x, S_q, S_k, S_v, S_ctx, S_r1, S_h1, S_gi, S_go, S_r2, S_out;
} ibert_layer_desc;

/* Uploads the parameters and precomputes every integer constant of the layer. */
int ibert_layer_create(ibert_ctx* ctx, const ibert_layer_desc* desc, ibert_layer** out);
int ibert_layer_destroy(ibert_layer* layer);

/* Linear layer, residual addition and i-LayerNorm as one operation -- the tail of both halves of
   the encoder layer (Fig. 1 right; Sec. 3.6, Eq. 16 on top of the integer linear layer):
     out = i-LayerNorm( requant_Q16(x w^T + bias, S_mid) + rescale(res, S_res -> S_mid) ; gamma, beta, S_out )
   x: device int8 [M, K]; w: device int8 [N, K] with host scales S_w[N]; bias: device int32 [N] at
   scale S_x*S_w[n], or NULL; res: device int8 [M, N] at host scale S_res; gamma, beta: host
   double [N]; out: device int8 [M, N] at S_out (*S_ret).  The result is bit-identical to
   ibert_linear_i8(kind 1, S_mid) followed by ibert_layernorm_i.  When N is a multiple of 256 (at
   most 1024), the constants fit the 32-bit forms and M is large enough for its 128-row tiles to
   occupy half of the SMs, a single kernel computes it on a cluster of N/256 CTAs per tile and the
   Q16 tensor never reaches memory; otherwise the two kernels run back to back through the
   context's workspace, which holds the Q16 tensor as int16.
   Errors: as ibert_linear_i8 and ibert_layernorm_i. */
int ibert_linear_layernorm_i8(ibert_ctx* ctx, const int8_t* x, double S_x, const int8_t* w, const double* S_w,
                              const int32_t* bias, int64_t M, int N, int K, double S_mid,
                              const int8_t* res, double S_res, const double* gamma, const double* beta,
                              double S_out, int8_t* out, double* S_ret);

/* How ibert_linear_layernorm_i8 and ibert_encoder_layer choose between the single cluster kernel and
   the two-kernel sequence (the results are identical): mode 0 (default) by problem size, 1 the
   cluster kernel whenever shapes and constants allow it, 2 never.  No counterpart in the paper:
   a tuning and testing switch.  Returns IBERT_ERR_ARG for another mode. */
int ibert_set_fusion(ibert_ctx* ctx, int mode);

/* How the linear layers (ibert_linear_i8, ibert_linear_gelu_i8, ibert_linear_hgelu_i8 and the GEMMs
   inside ibert_encoder_layer that are not taken by the cluster kernel above) treat problems with
   fewer 128 x 128 output tiles than SMs: mode 0 (default) splits K over a cluster of 2 or 4 CTAs
   per tile when that engages more SMs, 1 never splits, 2 and 4 force that width whenever K > 128.
   INT32 accumulation is exact, so the results are identical in every mode.  No counterpart in the
   paper: a tuning and testing switch.  Returns IBERT_ERR_ARG for another mode. */
int ibert_set_split_k(ibert_ctx* ctx, int mode);

/* How the FFN1 GEMM inside ibert_encoder_layer (CTA-pair tiles, i.e. large batches) evaluates
   i-GELU (Algorithm 2) and the requantization behind it: mode 0 (default) looks the int8 result up
   in a 65535-entry table over the Q16 input, which ibert_layer_create fills by running the
   i-GELU kernel over every Q16 value (64 KB of device memory per layer, copied into shared memory
   by every CTA); mode 1 computes it per element.  The results are identical.  The paper names tables only
   as the approach it avoids (Sec. 3.2: on-chip memory, look-up rate); here the table is filled by
   the integer algorithm itself and used only where the epilogue's integer pipe is the bound.  A tuning and testing switch.  Returns IBERT_ERR_ARG for another mode. */
int ibert_set_gelu_table(ibert_ctx* ctx, int mode);

/* Layout of the two tensors that never leave ibert_encoder_layer -- Q | K | V between the QKV GEMM
   and attention, and the FFN1 result between its GEMM and the fused FFN2 + LayerNorm kernel (the
   public calls always take and return [tokens][channels]): mode 0 (default) keeps them transposed,
   [channels][tokens], where the shapes allow (padded batches with L a multiple of 16; for the FFN1
   result also a token count that is a multiple of 16 and at least 4096, a tensor of at most half
   the L2 cache, and the table form of i-GELU and the fused kernel in use) -- the producing GEMM then writes each thread's 32 tokens of
   one channel as contiguous bytes instead of transposing them through shared memory, and the
   consuming kernel reads the tiles as MN-major operands; mode 1 keeps [tokens][channels] always;
   mode 2 is mode 0 without the lower bound on the token count (for tests: small problems then
   run the transposed forms too).  The results are identical.  No counterpart in the paper: a tuning and testing switch.  Returns
   IBERT_ERR_ARG for another mode. */
int ibert_set_qkv_layout(ibert_ctx* ctx, int mode);

/* The integer-only encoder layer (Fig. 1 right; post-LN order):
   QKV projection -> attention (i-softmax) -> output projection -> +x, i-LayerNorm ->
   FFN1 + i-GELU -> FFN2 -> +h1, i-LayerNorm.  x, out: int8 [B*L, H]; x at desc.S_x,
   out at desc.S_out (*S_ret).  Intermediates live in the context's workspace, which grows
   on demand (first call with a larger B*L allocates). */
int ibert_encoder_layer(ibert_ctx* ctx, const ibert_layer* layer, const int8_t* x, int B, int L,
                        int8_t* out, double* S_ret);

/* ---- around the plain layer: padded sequences, embedding, classifier -------------------------
   The paper treats none of these beyond stating that the Embedding is kept at INT8
   (implementation appendix); the readings below are this library's. */

/* Attention with a key-padding mask: lens (device int32 [B]) gives the valid keys of every
   sequence (values are clamped to [0, L]).  Keys j >= lens[b] take no part in the row maximum or
   the row sum of i-softmax (Algorithm 3) and get probability 0 -- the integer counterpart of an
   additive -inf mask; every query row, padded ones included, attends to the valid keys; a
   sequence without valid keys yields context 0.  Only the 32-key blocks that hold valid keys are
   computed.  Otherwise as ibert_attention_i8. */
int ibert_attention_masked_i8(ibert_ctx* ctx, const int8_t* qkv, int B, int L, int H, int heads,
                              const int32_t* lens, double S_q, double S_k, double S_v, double S_ctx, int p_max,
                              int8_t* out, double* S_ret);

/* ibert_encoder_layer on padded sequences: the attention step takes lens (device int32 [B]) as
   above; every other step is per token and runs on all B*L rows. */
int ibert_encoder_layer_masked(ibert_ctx* ctx, const ibert_layer* layer, const int8_t* x, int B, int L,
                               const int32_t* lens, int8_t* out, double* S_ret);

/* INT8 embedding + embedding LayerNorm: for token t (of T = B*L, row-major [B, L]),
     out[t, :] = i-LayerNorm( word[ids[t], :] + rescale(pos[t mod L, :], S_pos -> S_word) ; gamma, beta, S_out )
   i.e. the word row (int8 at S_word) is the LayerNorm input and the position row (int8 at S_pos)
   joins it as the residual does in ibert_layernorm_i (Sec. 3.6, Eq. 16).
   ids: device int32 [T] in [0, V) (an id outside records IBERT_ERR_VALUE_RANGE in the context's
   status and reads row 0); word: device int8 [V, H]; pos: device int8 [P, H], P >= L; gamma, beta:
   host double [H]; out: device int8 [T, H] at S_out.  H a multiple of 16, at most 2047.  Uses the
   context's workspace (5 bytes per element). */
int ibert_embedding_i8(ibert_ctx* ctx, const int32_t* ids, int64_t T, int L, const int8_t* word, int64_t V,
                       double S_word, const int8_t* pos, int64_t P, double S_pos, const double* gamma,
                       const double* beta, int H, double S_out, int8_t* out, double* S_ret);

/* Classifier head: one integer linear layer on the first token of every sequence,
     logits[b, n] = sum_k x[b*L, k] * w[n, k] + bias[n]          (raw INT32, scale S_x * S_w[n])
   x: device int8 [B*L, H]; w: device int8 [N, H] with host scales S_w[N]; bias: device int32 [N] or
   NULL; logits: device int32 [B, N]; S_ret (host, may be NULL) receives the N output scales.
   N a multiple of 4 (pad the label dimension with zero rows), H a multiple of 16. */
int ibert_classifier_i8(ibert_ctx* ctx, const int8_t* x, int B, int L, int H, double S_x, const int8_t* w,
                        const double* S_w, const int32_t* bias, int N, int32_t* logits, double* S_ret);

/* ---- packed batches: sequences of different lengths without padding ------------------------------
   The paper's workloads are sentence batches (GLUE), i.e. sequences of different lengths; it does
   not treat their layout.  Here a batch may be given PACKED: all tokens of all sequences in one
   [total_tokens, .] tensor, sequence b in rows cu_seqlens[b] .. cu_seqlens[b+1]-1 (cu_seqlens:
   device int32 [B + 1], non-decreasing, cu_seqlens[0] = 0, cu_seqlens[B] = total_tokens, every
   length at most max_len <= 512; total_tokens is passed on the host because it sizes the launches).
   Linear layers, i-GELU and i-LayerNorm are per token and simply run on total_tokens rows;
   attention (i-softmax, Algorithm 3) runs per sequence over its own rows.  The result for a
   sequence is the one ibert_encoder_layer_masked gives on its valid rows -- padding positions
   cost nothing instead of being computed and discarded.  A length above max_len records
   IBERT_ERR_VALUE_RANGE in the context's status (that sequence's surplus rows are not written).
   ibert_attention_packed_i8 returns IBERT_ERR_SCALE_RANGE for score scales so coarse that
   floor(ln2 / (S_q S_k / 8)) <= 2 (use the padded call there). */
int ibert_attention_packed_i8(ibert_ctx* ctx, const int8_t* qkv, const int32_t* cu_seqlens, int B, int max_len,
                              int64_t total_tokens, int H, int heads, double S_q, double S_k, double S_v,
                              double S_ctx, int p_max, int8_t* out, double* S_ret);
int ibert_encoder_layer_packed(ibert_ctx* ctx, const ibert_layer* layer, const int8_t* x, const int32_t* cu_seqlens,
                               int B, int max_len, int64_t total_tokens, int8_t* out, double* S_ret);
/* ibert_embedding_i8 on a packed batch: the position of a token is its distance from the first row
   of its sequence (P >= max_len).  ibert_classifier_i8 on a packed batch: the first token of
   sequence b is row cu_seqlens[b] (every sequence must have at least one token). */
int ibert_embedding_packed_i8(ibert_ctx* ctx, const int32_t* ids, const int32_t* cu_seqlens, int B, int max_len,
                              int64_t total_tokens, const int8_t* word, int64_t V, double S_word, const int8_t* pos,
                              int64_t P, double S_pos, const double* gamma, const double* beta, int H, double S_out,
                              int8_t* out, double* S_ret);
int ibert_classifier_packed_i8(ibert_ctx* ctx, const int8_t* x, const int32_t* cu_seqlens, int B, int H, double S_x,
                               const int8_t* w, const double* S_w, const int32_t* bias, int N, int32_t* logits,
                               double* S_ret);

/* ---- h-GELU, the comparison function of the paper (Eq. 6; Table 1, Table 3) --------------------
   h-GELU(x) = x ReLU6(1.702 x + 3) / 6.  The paper notes that it can be computed with integers
   but gives no integer algorithm; this library's reading keeps it parallel to i-GELU: the same
   integer q read at scale S_h = 1.702 S stands for 1.702 x, q_3 = floor(3 / S_h),
   q_6 = floor(6 / S_h), r = clamp(q + q_3, 0, q_6) >> s_h (s_h keeps the product in 32 bits),
   g = q r at scale S S_h 2^s_h / 6, then round(g / 256) and a dyadic requantization to int8.
   Not part of ibert_encoder_layer (the paper rejects h-GELU for its accuracy); provided to measure
   what i-GELU's polynomial costs.  Arguments, layouts and errors as ibert_gelu_i and
   ibert_linear_gelu_i8. */
int ibert_hgelu_i(ibert_ctx* ctx, const int32_t* q, double S, int64_t n, double S_out, int8_t* out,
                  double* S_ret);
int ibert_linear_hgelu_i8(ibert_ctx* ctx, const int8_t* x, double S_x, const int8_t* w, const double* S_w,
                          const int32_t* bias, int64_t M, int N, int K, double S_mid, double S_out,
                          int8_t* out, double* S_ret);

/* i-GELU by table look-up -- the alternative the paper argues against (Sec. 2, Sec. 3.4), here only
   for a measured comparison.  A 65535-entry int8 table for the scale pair (S, S_out) is built on
   first use by running the i-GELU kernel over every Q16 input (so its contents are Algorithm 2's
   results bit for bit) and cached in the context; afterwards each element costs one clamp and one
   load.  Results are identical to ibert_gelu_i.  Arguments and errors as ibert_gelu_i; the first
   call for a scale pair allocates 64 KiB of device memory (the context keeps at most 64 tables and
   drops them all, after synchronizing its stream, when a 65th is needed; ibert_destroy frees them). */
int ibert_gelu_lut_i(ibert_ctx* ctx, const int32_t* q, double S, int64_t n, double S_out, int8_t* out,
                     double* S_ret);

/* ---- a stack of encoder layers captured into a CUDA graph ---------------------------------------
   No counterpart in the paper: launch-overhead removal for small batches (a 12-layer pass is 60
   kernel launches).  ibert_encoder_graph_create runs layers[0..n_layers) once on the context's
   stream (x -> ... -> out, every layer with the same H; lens as in ibert_encoder_layer_masked or
   NULL) and captures the same sequence into a graph for these shapes and THESE buffers: a later
   ibert_encoder_graph_launch reads whatever x holds then and writes out.  The graph owns its
   workspace and intermediate activations (device memory allocated at creation, freed by
   ibert_encoder_graph_destroy, which synchronizes the stream first).  Creation fails with
   IBERT_ERR_ARG while ibert_profile_begin is active, and for a context created on the default
   stream (stream capture needs a stream of its own).  x, out, lens and the layers must stay alive
   and unmoved for the lifetime of the graph. */
typedef struct ibert_graph ibert_graph;
int ibert_encoder_graph_create(ibert_ctx* ctx, const ibert_layer* const* layers, int n_layers, const int8_t* x,
                               int B, int L, const int32_t* lens, int8_t* out, ibert_graph** graph);
int ibert_encoder_graph_launch(ibert_ctx* ctx, ibert_graph* graph);
int ibert_encoder_graph_destroy(ibert_graph* graph);

/* Per-kernel device timing (CUDA events recorded on the context's stream around every launch
   between begin and end).  No counterpart in the paper: measurement support only.
   ibert_profile_end synchronizes the stream and fills, per kernel class below, the summed
   device milliseconds and the number of launches (arrays of IBERT_NUM_KERNEL_CLASSES). */
enum {
  IBERT_K_GEMM_QKV = 0,      /* ibert_linear_i8 kind 0 / layer step QKV   */
  IBERT_K_ATTENTION = 1,
  IBERT_K_GEMM_Q16 = 2,      /* Q16 / raw epilogue with K <= 2048: output projection */
  IBERT_K_LAYERNORM = 3,
  IBERT_K_GEMM_GELU = 4,     /* FFN1 with fused i-GELU */
  IBERT_K_GEMM_Q16_WIDE = 5, /* Q16 / raw epilogue with K > 2048: FFN2 */
  IBERT_K_GELU = 6,
  IBERT_K_SOFTMAX = 7,
  IBERT_K_GEMM_LN = 8,       /* linear + residual + i-LayerNorm in one kernel, K <= 2048: output projection */
  IBERT_K_GEMM_LN_WIDE = 9,  /* the same with K > 2048: FFN2 */
  IBERT_NUM_KERNEL_CLASSES = 10
};
/* Host, pure.  Self-check of the constants derived from a score scale S for i-exp (Algorithm 3):
   verifies on the host, for every distance d in [0, 31*q_ln2] (and, for the unclamped form the
   attention kernel uses, every d < 2^21), that the multiply-high form the kernels use for
   z = floor(d / q_ln2) equals the division.  Returns IBERT_OK, the error of the
   derivation, or IBERT_ERR_VALUE_RANGE on a mismatch.  q_ln2_out (may be NULL) receives q_ln2. */
int ibert_selftest_exp_division(double S, int32_t* q_ln2_out);

/* Self-test of the bounded device-side waits (no counterpart in the paper): enqueues a two-warp
   kernel that waits on a barrier nobody arrives on -- one warp by the polling form of the wait,
   one by the form that parks the thread in hardware between polls (the GEMM feeder threads use
   it) -- with a limit of limit_us microseconds (1 .. 100000) on the GPU's nanosecond timer (the
   parked form may take up to about 20 ms longer).  When both limits have run out the kernel records
   IBERT_ERR_TIMEOUT in the context's status word -- exactly what every kernel of the library does
   when one of its waits (limit: one second) expires -- and returns normally; the context stays
   usable.  ibert_last_status() then returns IBERT_ERR_TIMEOUT once. */
int ibert_selftest_wait_timeout(ibert_ctx* ctx, int64_t limit_us);

int ibert_profile_begin(ibert_ctx* ctx);
int ibert_profile_end(ibert_ctx* ctx, float* ms, int32_t* launches);

#ifdef __cplusplus
}
#endif
#endif /* IBERT_H_ */
