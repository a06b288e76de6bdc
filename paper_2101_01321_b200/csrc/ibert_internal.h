// Internal declarations shared by the translation units of libibert_b200.
// Host-side constant derivation, the context object and the kernel launchers.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <map>
#include <vector>

#include "../../include/ibert.h"

namespace ibert {

// ---------------------------------------------------------------------------------------
// Integer constants the host derives from scales (kernels never see a floating-point value)
// ---------------------------------------------------------------------------------------

// i-exp / i-softmax (Algorithm 3).  S' = S * 2^s_in is the scale the polynomial works at.
struct ExpConsts {
  int32_t s_in;      // static pre-shift of the distance from the row maximum
  uint32_t q_ln2;    // floor(ln2 / S')
  uint32_t d_max;    // 31 * q_ln2: any larger distance gives e = 0
  // floor(d / q_ln2) = umulhi(d << div_pre, div_m) >> div_post, exact for every d <= d_max
  uint32_t div_m;
  int32_t div_pre, div_post;
  int32_t q_b;       // floor(1.353 / S')
  int32_t q_c;       // floor(0.344 / (0.3585 S'^2))
  int32_t s_out;     // static post-shift: every e < 2^21
  uint32_t p_max;    // 255 or 127: the fixed-point one of the probabilities
  // the same division for distances known to stay below 2^21 (scores of 64 int8 products):
  // floor(d / q_ln2) = umulhi(d, wide_m) >> wide_post for every d < 2^21, no clamp to d_max needed
  uint32_t wide_m;
  int32_t wide_post;
  // k when q_ln2 = 2^k and s_in = 0 (score scale exactly ln2 / 2^k): quotient and remainder of the
  // distance are then a shift and a mask; -1 otherwise
  int32_t pow2_k;
};

// i-GELU (Algorithm 2) followed by requantization to int8
struct GeluConsts {
  int32_t s_in;      // static pre-shift of the erf argument
  int32_t nq_b;      // -floor(-1.769 / S2) > 0: clip point of |q| and offset of the polynomial
  int32_t q_c;       // floor(1 / (-0.2888 S2^2)) < 0 (also q_1 = floor(1 / S_erf))
  int32_t s_f;       // shift keeping q * (q_erf + q_1) in 32 bits
  int32_t b, c;      // dyadic multiplier from the scale of round(g / 256) to S_out
  // the same requantization as one multiply-add whose upper word is the result:
  // (g2 * b + 2^(c-1)) >> c == (g2 * b2 + add2) >> 32 with b2 = b << (32-c); valid when fast != 0
  int32_t b2, fast;
  int64_t add2;
  // h-GELU (Eq. 6) through the same plumbing: hard != 0 and the fields above mean
  // nq_b = q_6 = floor(6 / S_h), q_c = q_3 = floor(3 / S_h), s_f = s_h, s_in unused (S_h = 1.702 S)
  int32_t hard;
  // i-GELU only: the most negative result provably stays above -127 (its magnitude is bounded by
  // the minimum of x erf-polynomial, about 0.17 in real units), so no lower clamp is needed
  int32_t low_free;
};

// residual add in front of i-LayerNorm
struct LnConsts {
  int32_t C;
  int32_t has_res;
  int32_t b_r, c_r;  // dyadic(S_r / S)
  int32_t c;         // common shift of the per-channel affine multipliers
  // upper-word forms with the *value* pre-shifted (it has the headroom, the 31-bit multiplier
  // has none): residual rescale as ((r << res_sh) * b_r + 2^31) >> 32 with res_sh = 32 - c_r when
  // res_fast; output as ((n << out_sh) * b_i + (B_i << out_sh)) >> 32 with out_sh = 32 - c when
  // out_fast (the B_i table then already holds the shifted addends)
  int32_t res_sh, res_fast;
  int32_t out_sh, out_fast;
  // the residual rescale in 32-bit arithmetic: (r * res_nb + res_nhalf) >> res_nc with a 24-bit multiplier,
  // offered (res_narrow != 0) only when the host has checked all 256 int8 values against the exact form
  int32_t res_nb, res_nc, res_nhalf, res_narrow;
};

int dyadic(double m, int32_t* b, int32_t* c);
int make_exp_consts(double S, int p_max, ExpConsts* k);
int make_gelu_consts(double S, double S_out, GeluConsts* k);
int make_hgelu_consts(double S, double S_out, GeluConsts* k);
// per-channel multipliers b_i (int32) and addends B_i (int64, rounding constant included)
int make_ln_tables(const double* gamma, const double* beta, int C, double S_out, LnConsts* k,
                   std::vector<int32_t>* b_i, std::vector<int64_t>* B_i);
int make_ln_residual(double S_r, double S, LnConsts* k);
// per-output-channel dyadic multipliers of a linear layer; S_out_cols (N entries) or S_out
int make_linear_tables(double S_x, const double* S_w, int N, const double* S_out_cols, double S_out,
                       std::vector<int32_t>* b, std::vector<int32_t>* c);

// ---------------------------------------------------------------------------------------
// Context
// ---------------------------------------------------------------------------------------

struct DeviceTable {
  void* ptr = nullptr;
  size_t bytes = 0;
  std::vector<unsigned char> host;   // the bytes that were uploaded: a hit must match them
};

}  // namespace ibert

// launch-time state the kernels' launchers keep per device (function attributes are per device)
constexpr int kMaxDevices = 64;

struct ibert_ctx {
  int device = 0;
  cudaStream_t stream = nullptr;
  int32_t* d_status = nullptr;       // first device-side error (0 = none)
  int num_sms = 0;
  int64_t l2_bytes = 0;             // size of the L2 cache
  // derived constant tables already on the device, keyed by a hash of their host bytes
  std::map<uint64_t, ibert::DeviceTable> tables;
  // look-up tables of ibert_gelu_lut_i, keyed by a hash of the GELU constants
  int splitk_mode = 0;     // see gemm_splitk_width
  std::map<uint64_t, int8_t*> gelu_luts;
  std::map<uint64_t, uint32_t*> exp_luts;
  // workspace for the encoder layer's intermediates
  void* ws = nullptr;
  size_t ws_bytes = 0;
  // linear + LayerNorm fusion: 0 = by problem size, 1 = whenever supported, 2 = never (ibert_set_fusion)
  int fusion_mode = 0;
  // i-GELU inside the large-tile GEMM epilogue: 0 = from the layer's table, 1 = computed (ibert_set_gelu_table)
  int gelu_table_mode = 0;
  // layout of the layer's internal Q | K | V tensor: 0 = transposed [3H][tokens] where the shapes allow it
  // (the QKV GEMM then needs no transposing store), 1 = always [tokens][3H] (ibert_set_qkv_layout)
  int qkv_layout_mode = 0;          // 0: transposed intermediates where they pay, 1: never, 2: wherever shapes allow
  // optional per-launch event timing (ibert_profile_begin / _end)
  bool profiling = false;
  std::vector<cudaEvent_t> ev_pool;      // pairs: [2i] before, [2i+1] after launch i
  std::vector<int> ev_class;             // kernel class of launch i
};

namespace ibert {

// uploads `bytes` of host data once per distinct content; returns the device copy
int cached_upload(ibert_ctx* ctx, const void* host, size_t bytes, uint64_t tag, void** dev);
int trim_tables(ibert_ctx* ctx);   // bounds the cache; only at the start of an entry point

// ---------------------------------------------------------------------------------------
// Kernel launchers (each returns an IBERT_* code; all enqueue on ctx->stream)
// ---------------------------------------------------------------------------------------

// one warp that waits `limit_ns` on a barrier nobody arrives on, then records IBERT_ERR_TIMEOUT
int launch_wait_timeout(ibert_ctx* ctx, uint64_t limit_ns);
int launch_gelu(ibert_ctx* ctx, const int32_t* q, int64_t n, const GeluConsts& k, int8_t* out);
// table[i] = i-GELU(i - 32767) for i in [0, 65535), computed by the i-GELU kernel over a ramp written
// to `ramp_scratch` (65535 int32); and the look-up kernel that uses it
int launch_gelu_table(ibert_ctx* ctx, const GeluConsts& k, int32_t* ramp_scratch, int8_t* table);
int launch_gelu_lut(ibert_ctx* ctx, const int32_t* q, int64_t n, const int8_t* table, int8_t* out);
int launch_softmax(ibert_ctx* ctx, const int32_t* q, int64_t rows, int L, const ExpConsts& k, uint8_t* out,
                   const uint32_t* exp_table = nullptr);
int launch_exp_table(ibert_ctx* ctx, const ExpConsts& k, uint32_t* table);
// rows of the word table (as int32) and of the position table (token t: position t mod L) gathered
// into q [T, H] and r [T, H]; an id outside [0, V) records IBERT_ERR_VALUE_RANGE and reads row 0
// (cu_seqlens != null: packed batch of B sequences, position = distance from the sequence's first row)
int launch_embed_gather(ibert_ctx* ctx, const int32_t* ids, int64_t T, int L, const int8_t* word, int64_t V,
                        const int8_t* pos, int H, int32_t* q, int8_t* r, const int32_t* cu_seqlens = nullptr,
                        int B = 0);
// out[b, :] = x[cu_seqlens[b], :] for b < B (first token of every sequence of a packed batch)
int launch_gather_first_rows(ibert_ctx* ctx, const int8_t* x, const int32_t* cu_seqlens, int B, int H, int8_t* out);
int launch_layernorm(ibert_ctx* ctx, const int32_t* q, const int8_t* r, int64_t rows, const LnConsts& k,
                     const int32_t* d_b, const int64_t* d_B, int8_t* out);
// the same with the Q16 input stored as int16 (values identical, 2 bytes per element less traffic)
int launch_layernorm_i16(ibert_ctx* ctx, const int16_t* q, const int8_t* r, int64_t rows, const LnConsts& k,
                         const int32_t* d_b, const int64_t* d_B, int8_t* out);

// epilogue kinds of the GEMM
// (EPI_Q16H: the Q16 values of EPI_Q16 stored as int16 instead of int32)
enum : int { EPI_INT8 = 0, EPI_Q16 = 1, EPI_RAW = 2, EPI_GELU = 3, EPI_HGELU = 4, EPI_Q16H = 5 };

struct GemmEpilogue {
  int kind;
  const int32_t* d_b;      // [N] dyadic multipliers b (fast: b << (32 - c)); unused for EPI_RAW
  const int32_t* d_c;      // [N] dyadic shifts
  const int32_t* d_bias;   // [N] or nullptr
  int fast;                // 1: every column's requantization fits the upper-word form; 2: the wide
                           // upper-word form (d_b = low words, d_c = integer parts; GELU epilogue of
                           // the plain GEMM only); 0: generic (b, c) pairs
  GeluConsts gelu;         // EPI_GELU / EPI_HGELU only
  // EPI_GELU, optional: table[i] = i-GELU(i - 32767) as int8 for every Q16 value (launch_gelu_table).
  // Tile shapes with 64 KB of shared memory to spare then look the result up instead of computing it.
  const int8_t* gelu_table = nullptr;
  // EPI_INT8 in the upper-word form only: the result is written TRANSPOSED, out[n][t] (M a multiple of 16).
  // A thread of the GEMM owns one channel and 32 tokens, so its results are contiguous bytes of the
  // transposed tensor and leave without a transposing store; the attention kernel reads that layout.
  bool out_transposed = false;
};

// Upper-word form of a column set: true if for every n, c[n] >= 1 and b[n] << (32 - c[n]) fits
// int32; then b is replaced by the shifted multipliers.
bool to_upper_word_form(std::vector<int32_t>* b, const std::vector<int32_t>& c);
// The same for multipliers of 1/2 and more: b <- low word r, c <- integer part w of b 2^(32-c) =
// w 2^32 + r; false (nothing changed) when a shift is 0 or |v| <= max_abs_v could overflow v w.
bool to_upper_word_wide(std::vector<int32_t>* b, std::vector<int32_t>* c, int64_t max_abs_v);

int launch_gemm_i8(ibert_ctx* ctx, const int8_t* x, const int8_t* w, int64_t M, int N, int K,
                   const GemmEpilogue& epi, void* out);

// Split-K variant for problems with fewer 128 x 128 output tiles than SMs: a cluster of `split`
// (2 or 4) CTAs per tile, each over 1/split of K, reduced through distributed shared memory.
// gemm_splitk_width returns the width worth using (1 = do not split); ctx->splitk_mode overrides
// it (0 = by size, 1 = never, 2 / 4 = that width whenever the shapes allow).
int gemm_splitk_width(const ibert_ctx* ctx, int64_t M, int N, int K);
int launch_gemm_splitk_i8(ibert_ctx* ctx, const int8_t* x, const int8_t* w, int64_t M, int N, int K,
                          const GemmEpilogue& epi, void* out, int split);

// Launch with programmatic stream serialization (the kernel must call grid_dep_wait() before its
// first global-memory access) and an optional cluster width.
template <typename... KArgs, typename... Args>
inline int launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                      int cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = cluster_x;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...) != cudaSuccess) {
    cudaGetLastError();
    return IBERT_ERR_CUDA;
  }
  return IBERT_OK;
}

struct AttnConsts {
  ExpConsts e;
  int32_t b, c;            // dyadic((1/p_max) * S_v / S_ctx)
  int32_t b2, fast;        // upper-word form: (v * b2 + 2^31) >> 32 with b2 = b << (32 - c)
};

// GEMM + residual + i-LayerNorm in one kernel (cluster of H / 256 CTAs per 128-token tile):
// out = LN(requant_Q16(x w^T + bias) + rescale(res)).  `gemm_ln_supported` tells whether the
// shapes and constants allow it; otherwise run launch_gemm_i8 (Q16) followed by launch_layernorm.
bool gemm_ln_supported(int H, int K, const GemmEpilogue& epi, const LnConsts& ln);
int launch_gemm_ln_i8(ibert_ctx* ctx, const int8_t* x, const int8_t* w, int64_t T, int H, int K,
                      const GemmEpilogue& epi, const int8_t* res, const LnConsts& ln, const int32_t* d_b_i,
                      const int64_t* d_B_i, int8_t* out, bool x_transposed = false);

// `lens` (device, [B], may be null): valid keys per sequence -- keys beyond take no part in the
// softmax and get probability 0 (key-padding mask)
// `cu_seqlens` (device, [B + 1], may be null): packed batch -- qkv and out are [total_rows, .] without
// padding, sequence b occupies rows cu_seqlens[b] .. cu_seqlens[b+1]-1 (at most L); lens is ignored
int launch_attention(ibert_ctx* ctx, const int8_t* qkv, int B, int L, int H, int heads,
                     const AttnConsts& k, const int32_t* lens, int8_t* out, const int32_t* cu_seqlens = nullptr,
                     int64_t total_rows = 0, bool qkv_t = false);
// true when launch_attention can read the transposed tensor qkv^T [3H][B L] (qkv_t): padded batch, L a
// multiple of 16, a score scale the main kernel takes
bool attention_takes_transposed(int B, int L, const AttnConsts& k);
// whether the table form of the FFN1 epilogue can write its result transposed for an [M, N] problem
bool gemm_gelu_takes_transposed(const ibert_ctx* ctx, int64_t M, int N);

}  // namespace ibert
