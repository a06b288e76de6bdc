// C-ABI entry points of libibert_b200: argument validation, constant derivation,
// launch.  No entry point synchronizes (except ibert_last_status) and none has a CPU path.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

#include "ibert_internal.h"

using namespace ibert;

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool good_scale(double s) { return std::isfinite(s) && s > 0.0; }

uint64_t fnv1a(const void* data, size_t bytes, uint64_t seed) {
  const unsigned char* p = static_cast<const unsigned char*>(data);
  uint64_t h = 1469598103934665603ull ^ seed;
  for (size_t i = 0; i < bytes; ++i) { h ^= p[i]; h *= 1099511628211ull; }
  return h;
}

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    ok = cudaGetDevice(&prev) == cudaSuccess;
    if (ok && prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

// Records an event pair around one launch while profiling is on.
struct ProfileScope {
  ibert_ctx* ctx;
  size_t slot = 0;
  bool on = false;
  ProfileScope(ibert_ctx* c, int kclass) : ctx(c) {
    if (!c->profiling) return;
    slot = c->ev_class.size();
    while (c->ev_pool.size() < 2 * (slot + 1)) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return;
      c->ev_pool.push_back(e);
    }
    c->ev_class.push_back(kclass);
    on = cudaEventRecord(c->ev_pool[2 * slot], c->stream) == cudaSuccess;
  }
  ~ProfileScope() {
    if (on) cudaEventRecord(ctx->ev_pool[2 * slot + 1], ctx->stream);
  }
};

// No exception leaves the C ABI: a failed host allocation becomes IBERT_ERR_NOMEM, anything else
// IBERT_ERR_ARG (nothing in the library throws on purpose).
template <typename F>
inline int guarded(F&& body) noexcept {
  try {
    return body();
  } catch (const std::bad_alloc&) {
    return IBERT_ERR_NOMEM;
  } catch (...) {
    return IBERT_ERR_ARG;
  }
}

inline int gemm_class(int kind, int K) {
  if (kind == EPI_INT8) return IBERT_K_GEMM_QKV;
  if (kind == EPI_GELU || kind == EPI_HGELU) return IBERT_K_GEMM_GELU;
  return K > 2048 ? IBERT_K_GEMM_Q16_WIDE : IBERT_K_GEMM_Q16;
}

}  // namespace

namespace ibert {

// Bounds the cache of constant tables: once it holds more than 4096 entries, everything is dropped
// after the stream has gone idle.  Called at the START of an entry point, before it looks anything
// up -- a call holds the pointers it got from the cache until its kernels are enqueued, so the
// cache must never shrink in the middle of one.
int trim_tables(ibert_ctx* ctx) {
  if (ctx->tables.size() <= 4096) return IBERT_OK;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return IBERT_ERR_CUDA;
  for (auto& kv : ctx->tables) cudaFree(kv.second.ptr);
  ctx->tables.clear();
  return IBERT_OK;
}

int cached_upload(ibert_ctx* ctx, const void* host, size_t bytes, uint64_t tag, void** dev) {
  const uint64_t key = fnv1a(host, bytes, tag * 0x9e3779b97f4a7c15ull + bytes);
  auto it = ctx->tables.find(key);
  if (it != ctx->tables.end()) {
    // the hash only finds the candidate; the bytes decide
    if (it->second.bytes == bytes && (bytes == 0 || std::memcmp(it->second.host.data(), host, bytes) == 0)) {
      *dev = it->second.ptr;
      return IBERT_OK;
    }
    // two different tables with one hash: the newer one replaces the older once the stream is idle
    if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return IBERT_ERR_CUDA;
    cudaFree(it->second.ptr);
    ctx->tables.erase(it);
  }
  void* d = nullptr;
  if (cudaMalloc(&d, bytes ? bytes : 16) != cudaSuccess) { cudaGetLastError(); return IBERT_ERR_NOMEM; }
  if (cudaMemcpyAsync(d, host, bytes, cudaMemcpyHostToDevice, ctx->stream) != cudaSuccess) {
    cudaFree(d);
    return IBERT_ERR_CUDA;
  }
  DeviceTable t;
  t.ptr = d;
  t.bytes = bytes;
  t.host.assign(static_cast<const unsigned char*>(host), static_cast<const unsigned char*>(host) + bytes);
  ctx->tables[key] = std::move(t);
  *dev = d;
  return IBERT_OK;
}

}  // namespace ibert

struct ibert_layer {
  ibert_ctx* ctx = nullptr;
  ibert_layer_desc d{};              // scalars only are meaningful after create
  int8_t *w_qkv = nullptr, *w_o = nullptr, *w_f1 = nullptr, *w_f2 = nullptr;
  int32_t *bias_qkv = nullptr, *bias_o = nullptr, *bias_f1 = nullptr, *bias_f2 = nullptr;
  int32_t *b_qkv = nullptr, *c_qkv = nullptr, *b_o = nullptr, *c_o = nullptr;
  int32_t *b_f1 = nullptr, *c_f1 = nullptr, *b_f2 = nullptr, *c_f2 = nullptr;
  int fast_qkv = 0, fast_o = 0, fast_f1 = 0, fast_f2 = 0;   // multipliers stored in upper-word form
  int32_t *ln1_b = nullptr, *ln2_b = nullptr;
  int64_t *ln1_B = nullptr, *ln2_B = nullptr;
  LnConsts ln1{}, ln2{};
  GeluConsts gelu{};
  int8_t* gelu_table = nullptr;      // i-GELU of every Q16 value (FFN1 epilogue), or null
  AttnConsts attn{};
  std::vector<void*> owned;
};

extern "C" {

const char* ibert_strerror(int code) {
  switch (code) {
    case IBERT_OK: return "ok";
    case IBERT_ERR_ARG: return "invalid argument";
    case IBERT_ERR_SHAPE: return "unsupported shape";
    case IBERT_ERR_SCALE_RANGE: return "scale out of range";
    case IBERT_ERR_ALIGN: return "pointer or pitch not 16-byte aligned";
    case IBERT_ERR_NOMEM: return "out of memory";
    case IBERT_ERR_CUDA: return "CUDA call failed";
    case IBERT_ERR_TIMEOUT: return "bounded device wait expired";
    case IBERT_ERR_VALUE_RANGE: return "integer value out of the assumed range";
    default: return "unknown error";
  }
}

int ibert_dyadic_from_double(double m, int32_t* b, int32_t* c) {
  return guarded([&]() -> int {
  if (!b || !c) return IBERT_ERR_ARG;
  return dyadic(m, b, c);
  });
}

int ibert_create(ibert_ctx** out, int device, void* cuda_stream) {
  return guarded([&]() -> int {
  if (!out) return IBERT_ERR_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
    cudaGetLastError();
    return IBERT_ERR_CUDA;
  }
  DeviceGuard guard(device);
  if (!guard.ok) return IBERT_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return IBERT_ERR_CUDA;
  if (prop.major != 10) return IBERT_ERR_CUDA;       // sm_100a kernels only
  ibert_ctx* ctx = new (std::nothrow) ibert_ctx();
  if (!ctx) return IBERT_ERR_NOMEM;
  ctx->device = device;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  ctx->num_sms = prop.multiProcessorCount;
  ctx->l2_bytes = prop.l2CacheSize;
  if (cudaMalloc(&ctx->d_status, 64) != cudaSuccess) { delete ctx; return IBERT_ERR_NOMEM; }
  if (cudaMemsetAsync(ctx->d_status, 0, 64, ctx->stream) != cudaSuccess) {
    cudaFree(ctx->d_status);
    delete ctx;
    return IBERT_ERR_CUDA;
  }
  *out = ctx;
  return IBERT_OK;
  });
}

int ibert_destroy(ibert_ctx* ctx) {
  return guarded([&]() -> int {
  if (!ctx) return IBERT_ERR_ARG;
  DeviceGuard guard(ctx->device);
  cudaStreamSynchronize(ctx->stream);
  for (auto& kv : ctx->tables) cudaFree(kv.second.ptr);
  for (auto& kv : ctx->gelu_luts) cudaFree(kv.second);
  for (auto& kv : ctx->exp_luts) cudaFree(kv.second);
  for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
  if (ctx->ws) cudaFree(ctx->ws);
  cudaFree(ctx->d_status);
  delete ctx;
  return IBERT_OK;
  });
}

int ibert_set_fusion(ibert_ctx* ctx, int mode) {
  return guarded([&]() -> int {
  if (!ctx || mode < 0 || mode > 2) return IBERT_ERR_ARG;
  ctx->fusion_mode = mode;
  return IBERT_OK;
  });
}

int ibert_set_split_k(ibert_ctx* ctx, int mode) {
  return guarded([&]() -> int {
  if (!ctx || (mode != 0 && mode != 1 && mode != 2 && mode != 4)) return IBERT_ERR_ARG;
  ctx->splitk_mode = mode;
  return IBERT_OK;
  });
}

int ibert_set_qkv_layout(ibert_ctx* ctx, int mode) {
  return guarded([&]() -> int {
  if (!ctx || mode < 0 || mode > 2) return IBERT_ERR_ARG;
  ctx->qkv_layout_mode = mode;
  return IBERT_OK;
  });
}

int ibert_set_gelu_table(ibert_ctx* ctx, int mode) {
  return guarded([&]() -> int {
  if (!ctx || mode < 0 || mode > 1) return IBERT_ERR_ARG;
  ctx->gelu_table_mode = mode;
  return IBERT_OK;
  });
}

int ibert_last_status(ibert_ctx* ctx) {
  return guarded([&]() -> int {
  if (!ctx) return IBERT_ERR_ARG;
  DeviceGuard guard(ctx->device);
  int32_t st = 0;
  if (cudaMemcpyAsync(&st, ctx->d_status, sizeof(st), cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess)
    return IBERT_ERR_CUDA;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return IBERT_ERR_CUDA;
  if (st != 0) cudaMemsetAsync(ctx->d_status, 0, sizeof(st), ctx->stream);
  return st;
  });
}

static int gelu_common(ibert_ctx* ctx, const int32_t* q, double S, int64_t n, double S_out, int8_t* out,
                       double* S_ret, bool hard) {
  if (!ctx || n < 0 || (n > 0 && (!q || !out))) return IBERT_ERR_ARG;
  if (!aligned16(q) || !aligned16(out)) return IBERT_ERR_ALIGN;
  GeluConsts k;
  int rc = hard ? make_hgelu_consts(S, S_out, &k) : make_gelu_consts(S, S_out, &k);
  if (rc) return rc;
  DeviceGuard guard(ctx->device);
  {
    ProfileScope ps(ctx, IBERT_K_GELU);
    rc = launch_gelu(ctx, q, n, k, out);
  }
  if (rc == IBERT_OK && S_ret) *S_ret = S_out;
  return rc;
}

int ibert_gelu_i(ibert_ctx* ctx, const int32_t* q, double S, int64_t n, double S_out, int8_t* out,
                 double* S_ret) {
  return guarded([&]() -> int {
  return gelu_common(ctx, q, S, n, S_out, out, S_ret, false);
  });
}

static int ensure_workspace(ibert_ctx* ctx, size_t need);

// The 65535-entry i-GELU table of one scale pair, cached in the context (built once: a ramp into the
// workspace, the i-GELU kernel over it).  The pointer stays valid until a later entry point trims the cache.
static int cached_gelu_table(ibert_ctx* ctx, const GeluConsts& k, const int8_t** out) {
  const uint64_t key = fnv1a(&k, sizeof(k), 0x6c7574ull);
  if (ctx->gelu_luts.size() >= 64) {                 // bounded: drop every table once the stream is idle
    if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return IBERT_ERR_CUDA;
    for (auto& kv : ctx->gelu_luts) cudaFree(kv.second);
    ctx->gelu_luts.clear();
  }
  auto it = ctx->gelu_luts.find(key);
  if (it != ctx->gelu_luts.end()) { *out = it->second; return IBERT_OK; }
  int8_t* table = nullptr;
  if (int rc = ensure_workspace(ctx, 65536 * sizeof(int32_t))) return rc;
  if (cudaMalloc((void**)&table, 65536) != cudaSuccess) { cudaGetLastError(); return IBERT_ERR_NOMEM; }
  if (int rc = launch_gelu_table(ctx, k, static_cast<int32_t*>(ctx->ws), table)) { cudaFree(table); return rc; }
  ctx->gelu_luts[key] = table;
  *out = table;
  return IBERT_OK;
}

int ibert_gelu_lut_i(ibert_ctx* ctx, const int32_t* q, double S, int64_t n, double S_out, int8_t* out,
                     double* S_ret) {
  return guarded([&]() -> int {
  if (!ctx || n < 0 || (n > 0 && (!q || !out))) return IBERT_ERR_ARG;
  if (!aligned16(q) || !aligned16(out)) return IBERT_ERR_ALIGN;
  GeluConsts k{};                                   // zeroed: the bytes are hashed below
  int rc = make_gelu_consts(S, S_out, &k);
  if (rc) return rc;
  DeviceGuard guard(ctx->device);
  const int8_t* table = nullptr;
  if ((rc = cached_gelu_table(ctx, k, &table))) return rc;
  {
    ProfileScope ps(ctx, IBERT_K_GELU);
    rc = launch_gelu_lut(ctx, q, n, table, out);
  }
  if (rc == IBERT_OK && S_ret) *S_ret = S_out;
  return rc;
  });
}

int ibert_hgelu_i(ibert_ctx* ctx, const int32_t* q, double S, int64_t n, double S_out, int8_t* out,
                  double* S_ret) {
  return guarded([&]() -> int {
  return gelu_common(ctx, q, S, n, S_out, out, S_ret, true);
  });
}

static int softmax_common(ibert_ctx* ctx, const int32_t* q, double S, int64_t rows, int L, int p_max,
                          uint8_t* out, double* S_ret, bool by_table) {
  if (!ctx || rows < 0) return IBERT_ERR_ARG;
  if (p_max != 255 && p_max != 127) return IBERT_ERR_ARG;
  if (L < 1 || L > 1024) return IBERT_ERR_SHAPE;
  if (rows > 0 && (!q || !out)) return IBERT_ERR_ARG;
  if (!aligned16(q) || !aligned16(out)) return IBERT_ERR_ALIGN;
  ExpConsts k{};                                    // zeroed: the bytes are hashed below
  int rc = make_exp_consts(S, p_max, &k);
  if (rc) return rc;
  DeviceGuard guard(ctx->device);
  uint32_t* table = nullptr;
  if (by_table) {
    const uint64_t key = fnv1a(&k, sizeof(k), 0x657870ull);
    if (ctx->exp_luts.size() >= 64) {                // bounded: drop every table once the stream is idle
      if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return IBERT_ERR_CUDA;
      for (auto& kv : ctx->exp_luts) cudaFree(kv.second);
      ctx->exp_luts.clear();
    }
    auto it = ctx->exp_luts.find(key);
    if (it != ctx->exp_luts.end()) table = it->second;
    else {
      // built once per scale: the i-exp of every pre-shifted distance 0 .. d_max
      if (cudaMalloc((void**)&table, ((size_t)k.d_max + 1) * sizeof(uint32_t)) != cudaSuccess) {
        cudaGetLastError();
        return IBERT_ERR_NOMEM;
      }
      if ((rc = launch_exp_table(ctx, k, table))) { cudaFree(table); return rc; }
      ctx->exp_luts[key] = table;
    }
  }
  {
    ProfileScope ps(ctx, IBERT_K_SOFTMAX);
    rc = launch_softmax(ctx, q, rows, L, k, out, table);
  }
  if (rc == IBERT_OK && S_ret) *S_ret = 1.0 / (double)p_max;
  return rc;
}

int ibert_softmax_i(ibert_ctx* ctx, const int32_t* q, double S, int64_t rows, int L, int p_max,
                    uint8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  return softmax_common(ctx, q, S, rows, L, p_max, out, S_ret, false);
  });
}

int ibert_softmax_lut_i(ibert_ctx* ctx, const int32_t* q, double S, int64_t rows, int L, int p_max,
                        uint8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  return softmax_common(ctx, q, S, rows, L, p_max, out, S_ret, true);
  });
}

static int layernorm_common(ibert_ctx* ctx, const void* q, bool q_is_i16, double S, const int8_t* r, double S_r,
                            const double* gamma, const double* beta, int64_t rows, int C, double S_out,
                            int8_t* out, double* S_ret) {
  if (!ctx || rows < 0 || !gamma || !beta) return IBERT_ERR_ARG;
  if (C < 1 || C > 2047) return IBERT_ERR_SHAPE;
  if (rows > 0 && (!q || !out)) return IBERT_ERR_ARG;
  if (!aligned16(q) || !aligned16(out) || (r && !aligned16(r))) return IBERT_ERR_ALIGN;
  if (!good_scale(S) || !good_scale(S_out)) return IBERT_ERR_SCALE_RANGE;
  LnConsts k{};
  k.C = C;
  k.has_res = r != nullptr;
  if (r) {
    int rc = make_ln_residual(S_r, S, &k);
    if (rc) return rc;
  }
  std::vector<int32_t> b_i;
  std::vector<int64_t> B_i;
  int rc = make_ln_tables(gamma, beta, C, S_out, &k, &b_i, &B_i);
  if (rc) return rc;
  DeviceGuard guard(ctx->device);
  if ((rc = trim_tables(ctx))) return rc;
  void *d_b = nullptr, *d_B = nullptr;
  rc = cached_upload(ctx, b_i.data(), b_i.size() * sizeof(int32_t), 11, &d_b);
  if (rc) return rc;
  rc = cached_upload(ctx, B_i.data(), B_i.size() * sizeof(int64_t), 12, &d_B);
  if (rc) return rc;
  {
    ProfileScope ps(ctx, IBERT_K_LAYERNORM);
    if (q_is_i16)
      rc = launch_layernorm_i16(ctx, static_cast<const int16_t*>(q), r, rows, k, (const int32_t*)d_b, (const int64_t*)d_B, out);
    else
      rc = launch_layernorm(ctx, static_cast<const int32_t*>(q), r, rows, k, (const int32_t*)d_b, (const int64_t*)d_B, out);
  }
  if (rc == IBERT_OK && S_ret) *S_ret = S_out;
  return rc;
}

int ibert_layernorm_i(ibert_ctx* ctx, const int32_t* q, double S, const int8_t* r, double S_r,
                      const double* gamma, const double* beta, int64_t rows, int C, double S_out,
                      int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  return layernorm_common(ctx, q, false, S, r, S_r, gamma, beta, rows, C, S_out, out, S_ret);
  });
}

int ibert_layernorm_i16(ibert_ctx* ctx, const int16_t* q, double S, const int8_t* r, double S_r,
                        const double* gamma, const double* beta, int64_t rows, int C, double S_out,
                        int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  return layernorm_common(ctx, q, true, S, r, S_r, gamma, beta, rows, C, S_out, out, S_ret);
  });
}

static int linear_common(ibert_ctx* ctx, const int8_t* x, double S_x, const int8_t* w, const double* S_w,
                         const int32_t* bias, int64_t M, int N, int K, int kind, double S_mid,
                         double S_out, void* out, double* S_ret) {
  if (!ctx || M < 0 || !S_w) return IBERT_ERR_ARG;
  if (kind < 0 || kind > 5) return IBERT_ERR_ARG;
  if (N < 1 || K < 1 || K % 16 != 0 || N % 4 != 0) return IBERT_ERR_SHAPE;
  if (kind == EPI_Q16H && N % 8 != 0) return IBERT_ERR_SHAPE;      // 16-byte aligned int16 rows
  if ((kind == EPI_INT8 || kind == EPI_GELU || kind == EPI_HGELU) && N % 16 != 0) return IBERT_ERR_SHAPE;
  if ((int64_t)K * 127 * 127 >= (int64_t(1) << 31)) return IBERT_ERR_SHAPE;
  if (M >= (int64_t(1) << 31) - 256) return IBERT_ERR_SHAPE;      // tile coordinates are 32-bit
  if (M > 0 && (!x || !out)) return IBERT_ERR_ARG;
  if (!w) return IBERT_ERR_ARG;
  if (!aligned16(x) || !aligned16(w) || !aligned16(out) || (bias && !aligned16(bias))) return IBERT_ERR_ALIGN;
  if (!good_scale(S_x)) return IBERT_ERR_SCALE_RANGE;
  for (int n = 0; n < N; ++n)
    if (!good_scale(S_w[n])) return IBERT_ERR_SCALE_RANGE;
  GemmEpilogue epi{};
  epi.kind = kind;
  epi.d_bias = bias;
  DeviceGuard guard(ctx->device);
  if (int rc = trim_tables(ctx)) return rc;
  if (kind != EPI_RAW) {
    const double S_acc_to = (kind == EPI_GELU || kind == EPI_HGELU) ? S_mid : S_out;
    std::vector<int32_t> b, c;
    int rc = make_linear_tables(S_x, S_w, N, nullptr, S_acc_to, &b, &c);
    if (rc) return rc;
    // The epilogue runs in ONE form: the upper-word form needs the per-channel multipliers AND (for
    // the GELU kinds) the final multiplier to fit it.  The per-channel table is converted only then --
    // the generic epilogue reads the plain (b, c) pairs.
    bool upper_ok = true;
    if (kind == EPI_GELU || kind == EPI_HGELU) {
      rc = kind == EPI_HGELU ? make_hgelu_consts(S_mid, S_out, &epi.gelu) : make_gelu_consts(S_mid, S_out, &epi.gelu);
      if (rc) return rc;
      upper_ok = epi.gelu.fast != 0;
    }
    epi.fast = (upper_ok && to_upper_word_form(&b, c)) ? 1 : 0;
    // i-GELU by table (the tile shapes with room for it use it)
    if (kind == EPI_GELU && epi.fast && ctx->gelu_table_mode == 0)
      if ((rc = cached_gelu_table(ctx, epi.gelu, &epi.gelu_table))) return rc;
    void *d_b = nullptr, *d_c = nullptr;
    rc = cached_upload(ctx, b.data(), b.size() * sizeof(int32_t), 21, &d_b);
    if (rc) return rc;
    rc = cached_upload(ctx, c.data(), c.size() * sizeof(int32_t), 22, &d_c);
    if (rc) return rc;
    epi.d_b = (const int32_t*)d_b;
    epi.d_c = (const int32_t*)d_c;
  }
  int rc;
  {
    ProfileScope ps(ctx, gemm_class(kind, K));
    rc = launch_gemm_i8(ctx, x, w, M, N, K, epi, out);
  }
  if (rc == IBERT_OK && S_ret) {
    if (kind == EPI_RAW) for (int n = 0; n < N; ++n) S_ret[n] = S_x * S_w[n];
    else *S_ret = S_out;
  }
  return rc;
}

// true when T tokens give the fused GEMM + LayerNorm kernel (one cluster of H / 256 CTAs per
// 128-token tile) enough tiles to occupy at least half of the SMs; measured crossover on config 2:
// the two-kernel path wins up to T = 2048 (0.63 vs 0.76 ms at T = 128), the fused one from T = 4096
static bool gemm_ln_profitable(const ibert_ctx* ctx, int64_t T, int H) {
  if (ctx->fusion_mode == 1) return true;
  if (ctx->fusion_mode == 2) return false;
  const int64_t tiles = (T + 127) / 128;
  return tiles * (H / 256) * 2 >= ctx->num_sms;
}

// grows the context's workspace to at least `need` bytes (stream-synchronizing reallocation)
static int ensure_workspace(ibert_ctx* ctx, size_t need) {
  if (need <= ctx->ws_bytes) return IBERT_OK;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return IBERT_ERR_CUDA;
  if (ctx->ws) cudaFree(ctx->ws);
  ctx->ws = nullptr;
  ctx->ws_bytes = 0;
  if (cudaMalloc(&ctx->ws, need) != cudaSuccess) { cudaGetLastError(); return IBERT_ERR_NOMEM; }
  ctx->ws_bytes = need;
  return IBERT_OK;
}

int ibert_linear_layernorm_i8(ibert_ctx* ctx, const int8_t* x, double S_x, const int8_t* w, const double* S_w,
                              const int32_t* bias, int64_t M, int N, int K, double S_mid,
                              const int8_t* res, double S_res, const double* gamma, const double* beta,
                              double S_out, int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  if (!ctx || M < 0 || !S_w || !gamma || !beta || !w) return IBERT_ERR_ARG;
  if (N < 1 || N > 2047 || K < 1 || K % 16 != 0 || N % 16 != 0) return IBERT_ERR_SHAPE;
  if ((int64_t)K * 127 * 127 >= (int64_t(1) << 31)) return IBERT_ERR_SHAPE;
  if (M >= (int64_t(1) << 31) - 256) return IBERT_ERR_SHAPE;      // tile coordinates are 32-bit
  if (M > 0 && (!x || !out || !res)) return IBERT_ERR_ARG;
  if (!aligned16(x) || !aligned16(w) || !aligned16(out) || !aligned16(res) || (bias && !aligned16(bias)))
    return IBERT_ERR_ALIGN;
  if (!good_scale(S_x) || !good_scale(S_mid) || !good_scale(S_out)) return IBERT_ERR_SCALE_RANGE;
  for (int n = 0; n < N; ++n)
    if (!good_scale(S_w[n])) return IBERT_ERR_SCALE_RANGE;
  GemmEpilogue epi{};
  epi.kind = EPI_Q16;
  epi.d_bias = bias;
  std::vector<int32_t> b, c;
  int rc = make_linear_tables(S_x, S_w, N, nullptr, S_mid, &b, &c);
  if (rc) return rc;
  epi.fast = to_upper_word_form(&b, c) ? 1 : 0;
  LnConsts k{};
  k.C = N;
  k.has_res = 1;
  rc = make_ln_residual(S_res, S_mid, &k);
  if (rc) return rc;
  std::vector<int32_t> b_i;
  std::vector<int64_t> B_i;
  rc = make_ln_tables(gamma, beta, N, S_out, &k, &b_i, &B_i);
  if (rc) return rc;
  DeviceGuard guard(ctx->device);
  if ((rc = trim_tables(ctx))) return rc;
  void *d_b = nullptr, *d_c = nullptr, *d_bi = nullptr, *d_Bi = nullptr;
  if ((rc = cached_upload(ctx, b.data(), b.size() * sizeof(int32_t), 21, &d_b))) return rc;
  if ((rc = cached_upload(ctx, c.data(), c.size() * sizeof(int32_t), 22, &d_c))) return rc;
  if ((rc = cached_upload(ctx, b_i.data(), b_i.size() * sizeof(int32_t), 11, &d_bi))) return rc;
  if ((rc = cached_upload(ctx, B_i.data(), B_i.size() * sizeof(int64_t), 12, &d_Bi))) return rc;
  epi.d_b = (const int32_t*)d_b;
  epi.d_c = (const int32_t*)d_c;
  if (gemm_ln_profitable(ctx, M, N) && gemm_ln_supported(N, K, epi, k)) {
    ProfileScope ps(ctx, K > 2048 ? IBERT_K_GEMM_LN_WIDE : IBERT_K_GEMM_LN);
    rc = launch_gemm_ln_i8(ctx, x, w, M, N, K, epi, res, k, (const int32_t*)d_bi, (const int64_t*)d_Bi, out);
  } else {
    // the Q16 tensor between the two kernels is held as int16 (value-identical, half the bytes)
    if ((rc = ensure_workspace(ctx, (size_t)M * N * 2 + 256))) return rc;
    int16_t* mid = static_cast<int16_t*>(ctx->ws);
    epi.kind = EPI_Q16H;
    { ProfileScope ps(ctx, gemm_class(EPI_Q16, K)); rc = launch_gemm_i8(ctx, x, w, M, N, K, epi, mid); }
    if (rc) return rc;
    ProfileScope ps(ctx, IBERT_K_LAYERNORM);
    rc = launch_layernorm_i16(ctx, mid, res, M, k, (const int32_t*)d_bi, (const int64_t*)d_Bi, out);
  }
  if (rc == IBERT_OK && S_ret) *S_ret = S_out;
  return rc;
  });
}

int ibert_linear_i8(ibert_ctx* ctx, const int8_t* x, double S_x, const int8_t* w, const double* S_w,
                    const int32_t* bias, int64_t M, int N, int K, int out_kind, double S_out,
                    void* out, double* S_ret) {
  return guarded([&]() -> int {
  if (out_kind < 0 || out_kind > 3) return IBERT_ERR_ARG;
  return linear_common(ctx, x, S_x, w, S_w, bias, M, N, K, out_kind == 3 ? (int)EPI_Q16H : out_kind, 0.0, S_out, out,
                       S_ret);
  });
}

int ibert_linear_gelu_i8(ibert_ctx* ctx, const int8_t* x, double S_x, const int8_t* w, const double* S_w,
                         const int32_t* bias, int64_t M, int N, int K, double S_mid, double S_out,
                         int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  return linear_common(ctx, x, S_x, w, S_w, bias, M, N, K, EPI_GELU, S_mid, S_out, out, S_ret);
  });
}

int ibert_linear_hgelu_i8(ibert_ctx* ctx, const int8_t* x, double S_x, const int8_t* w, const double* S_w,
                          const int32_t* bias, int64_t M, int N, int K, double S_mid, double S_out,
                          int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  return linear_common(ctx, x, S_x, w, S_w, bias, M, N, K, EPI_HGELU, S_mid, S_out, out, S_ret);
  });
}

static int make_attn_consts(double S_q, double S_k, double S_v, double S_ctx, int p_max, AttnConsts* k) {
  if (!good_scale(S_q) || !good_scale(S_k) || !good_scale(S_v) || !good_scale(S_ctx)) return IBERT_ERR_SCALE_RANGE;
  if (p_max != 255 && p_max != 127) return IBERT_ERR_ARG;
  int rc = make_exp_consts((S_q * S_k) / 8.0, p_max, &k->e);     // 1/sqrt(64) folded into the score scale
  if (rc) return rc;
  rc = dyadic(((1.0 / (double)p_max) * S_v) / S_ctx, &k->b, &k->c);
  if (rc) return rc;
  std::vector<int32_t> b1(1, k->b), c1(1, k->c);
  k->fast = to_upper_word_form(&b1, c1) ? 1 : 0;
  k->b2 = k->fast ? b1[0] : 0;
  return IBERT_OK;
}

static int attention_common(ibert_ctx* ctx, const int8_t* qkv, int B, int L, int H, int heads, const int32_t* lens,
                            double S_q, double S_k, double S_v, double S_ctx, int p_max, int8_t* out,
                            double* S_ret) {
  if (!ctx || B < 0) return IBERT_ERR_ARG;
  if (heads < 1 || H != heads * 64 || L < 1 || L > 512) return IBERT_ERR_SHAPE;
  if (B > 0 && (!qkv || !out)) return IBERT_ERR_ARG;
  if (!aligned16(qkv) || !aligned16(out)) return IBERT_ERR_ALIGN;
  AttnConsts k{};
  int rc = make_attn_consts(S_q, S_k, S_v, S_ctx, p_max, &k);
  if (rc) return rc;
  DeviceGuard guard(ctx->device);
  {
    ProfileScope ps(ctx, IBERT_K_ATTENTION);
    rc = launch_attention(ctx, qkv, B, L, H, heads, k, lens, out);
  }
  if (rc == IBERT_OK && S_ret) *S_ret = S_ctx;
  return rc;
}

int ibert_attention_i8(ibert_ctx* ctx, const int8_t* qkv, int B, int L, int H, int heads, double S_q,
                       double S_k, double S_v, double S_ctx, int p_max, int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  return attention_common(ctx, qkv, B, L, H, heads, nullptr, S_q, S_k, S_v, S_ctx, p_max, out, S_ret);
  });
}

int ibert_attention_masked_i8(ibert_ctx* ctx, const int8_t* qkv, int B, int L, int H, int heads,
                              const int32_t* lens, double S_q, double S_k, double S_v, double S_ctx, int p_max,
                              int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  if (B > 0 && !lens) return IBERT_ERR_ARG;
  return attention_common(ctx, qkv, B, L, H, heads, lens, S_q, S_k, S_v, S_ctx, p_max, out, S_ret);
  });
}

// --------------------------------------------------------------------------- encoder layer

static int upload_owned(ibert_layer* ly, const void* host, size_t bytes, void** dev) {
  void* d = nullptr;
  if (cudaMalloc(&d, bytes) != cudaSuccess) { cudaGetLastError(); return IBERT_ERR_NOMEM; }
  ly->owned.push_back(d);
  if (cudaMemcpyAsync(d, host, bytes, cudaMemcpyHostToDevice, ly->ctx->stream) != cudaSuccess) return IBERT_ERR_CUDA;
  *dev = d;
  return IBERT_OK;
}

int ibert_layer_destroy(ibert_layer* ly) {
  return guarded([&]() -> int {
  if (!ly) return IBERT_ERR_ARG;
  DeviceGuard guard(ly->ctx->device);
  cudaStreamSynchronize(ly->ctx->stream);
  for (void* p : ly->owned) cudaFree(p);
  delete ly;
  return IBERT_OK;
  });
}

int ibert_layer_create(ibert_ctx* ctx, const ibert_layer_desc* d, ibert_layer** out) {
  return guarded([&]() -> int {
  if (!ctx || !d || !out) return IBERT_ERR_ARG;
  *out = nullptr;
  const int H = d->H, F = d->F;
  if (d->heads < 1 || H != d->heads * 64 || F < 16 || F % 16 != 0) return IBERT_ERR_SHAPE;
  if (H > 2047) return IBERT_ERR_SHAPE;
  if ((int64_t)F * 127 * 127 >= (int64_t(1) << 31)) return IBERT_ERR_SHAPE;
  const void* ptrs[] = {d->w_qkv, d->S_w_qkv, d->bias_qkv, d->w_o, d->S_w_o, d->bias_o, d->w_f1, d->S_w_f1,
                        d->bias_f1, d->w_f2, d->S_w_f2, d->bias_f2, d->gamma1, d->beta1, d->gamma2, d->beta2};
  for (const void* p : ptrs) if (!p) return IBERT_ERR_ARG;
  const double scales[] = {d->S_x, d->S_q, d->S_k, d->S_v, d->S_ctx, d->S_r1, d->S_h1, d->S_gi, d->S_go, d->S_r2, d->S_out};
  for (double s : scales) if (!good_scale(s)) return IBERT_ERR_SCALE_RANGE;

  DeviceGuard guard(ctx->device);
  ibert_layer* ly = new (std::nothrow) ibert_layer();
  if (!ly) return IBERT_ERR_NOMEM;
  ly->ctx = ctx;
  // frees the half-built layer on every early exit, an exception included
  struct Holder {
    ibert_layer* p;
    ~Holder() { if (p) ibert_layer_destroy(p); }
  } holder{ly};
  ly->d = *d;
  int rc = IBERT_OK;
  auto up = [&](const void* h, size_t bytes, void** dev) { if (rc == IBERT_OK) rc = upload_owned(ly, h, bytes, dev); };
  // `upper_ok`: whether the rest of that GEMM's epilogue can run in the upper-word form; the table
  // is converted to it only then (the generic epilogue reads the plain (b, c) pairs)
  // `max_acc` > 0: the largest accumulator magnitude this GEMM can produce (K 127^2 + max |bias|); a
  // table that does not fit the upper-word form may then take the wide one (GELU epilogue only)
  auto lin = [&](double S_in, const double* S_w, int N, const double* so_cols, double so, int32_t** db, int32_t** dc,
                 int* fast, bool upper_ok = true, int64_t max_acc = 0) {
    if (rc != IBERT_OK) return;
    std::vector<int32_t> b, c;
    rc = make_linear_tables(S_in, S_w, N, so_cols, so, &b, &c);
    if (rc != IBERT_OK) return;
    *fast = (upper_ok && to_upper_word_form(&b, c)) ? 1 : 0;
    if (!*fast && upper_ok && max_acc > 0 && to_upper_word_wide(&b, &c, max_acc)) *fast = 2;
    up(b.data(), b.size() * sizeof(int32_t), (void**)db);
    up(c.data(), c.size() * sizeof(int32_t), (void**)dc);
  };
  up(d->w_qkv, (size_t)3 * H * H, (void**)&ly->w_qkv);
  up(d->w_o, (size_t)H * H, (void**)&ly->w_o);
  up(d->w_f1, (size_t)F * H, (void**)&ly->w_f1);
  up(d->w_f2, (size_t)H * F, (void**)&ly->w_f2);
  up(d->bias_qkv, sizeof(int32_t) * 3 * H, (void**)&ly->bias_qkv);
  up(d->bias_o, sizeof(int32_t) * H, (void**)&ly->bias_o);
  up(d->bias_f1, sizeof(int32_t) * F, (void**)&ly->bias_f1);
  up(d->bias_f2, sizeof(int32_t) * H, (void**)&ly->bias_f2);
  {
    std::vector<double> so(3 * (size_t)H);
    for (int n = 0; n < 3 * H; ++n) so[n] = n < H ? d->S_q : (n < 2 * H ? d->S_k : d->S_v);
    lin(d->S_x, d->S_w_qkv, 3 * H, so.data(), 0.0, &ly->b_qkv, &ly->c_qkv, &ly->fast_qkv);
  }
  lin(d->S_ctx, d->S_w_o, H, nullptr, d->S_r1, &ly->b_o, &ly->c_o, &ly->fast_o);
  if (rc == IBERT_OK) rc = make_gelu_consts(d->S_gi, d->S_go, &ly->gelu);
  int64_t max_acc_f1 = (int64_t)H * 127 * 127;
  {
    int64_t bmax = 0;
    for (int n = 0; n < F; ++n) bmax = std::max<int64_t>(bmax, std::llabs((int64_t)d->bias_f1[n]));
    max_acc_f1 += bmax;
  }
  lin(d->S_h1, d->S_w_f1, F, nullptr, d->S_gi, &ly->b_f1, &ly->c_f1, &ly->fast_f1, ly->gelu.fast != 0, max_acc_f1);
  lin(d->S_go, d->S_w_f2, H, nullptr, d->S_r2, &ly->b_f2, &ly->c_f2, &ly->fast_f2);
  auto ln = [&](const double* g, const double* be, double S_sum, double S_res, double S_o, LnConsts* k,
                int32_t** db, int64_t** dB) {
    if (rc != IBERT_OK) return;
    k->C = H;
    k->has_res = 1;
    rc = make_ln_residual(S_res, S_sum, k);
    if (rc != IBERT_OK) return;
    std::vector<int32_t> b_i;
    std::vector<int64_t> B_i;
    rc = make_ln_tables(g, be, H, S_o, k, &b_i, &B_i);
    up(b_i.data(), b_i.size() * sizeof(int32_t), (void**)db);
    up(B_i.data(), B_i.size() * sizeof(int64_t), (void**)dB);
  };
  ln(d->gamma1, d->beta1, d->S_r1, d->S_x, d->S_h1, &ly->ln1, &ly->ln1_b, &ly->ln1_B);
  ln(d->gamma2, d->beta2, d->S_r2, d->S_h1, d->S_out, &ly->ln2, &ly->ln2_b, &ly->ln2_B);
  if (rc == IBERT_OK) rc = make_attn_consts(d->S_q, d->S_k, d->S_v, d->S_ctx, d->p_max, &ly->attn);
  if (rc != IBERT_OK) return rc;
  // FFN1's i-GELU as a table over all Q16 inputs, written by the i-GELU kernel itself (the large-tile
  // GEMM looks results up in it; needs the upper-word form of the requantization in front of it)
  void* ramp = nullptr;
  if (ly->fast_f1 != 0 && ly->gelu.fast != 0) {
    void* t = nullptr;
    if (cudaMalloc(&t, 65536) != cudaSuccess || cudaMalloc(&ramp, 65536 * sizeof(int32_t)) != cudaSuccess) {
      cudaGetLastError();
      cudaFree(t);
      return IBERT_ERR_NOMEM;
    }
    ly->owned.push_back(t);
    rc = launch_gelu_table(ctx, ly->gelu, static_cast<int32_t*>(ramp), static_cast<int8_t*>(t));
    if (rc == IBERT_OK) ly->gelu_table = static_cast<int8_t*>(t);
  }
  // host arrays were pageable: make sure the copies have left them before returning
  const bool synced = cudaStreamSynchronize(ctx->stream) == cudaSuccess;
  cudaFree(ramp);
  if (rc != IBERT_OK) return rc;
  if (!synced) return IBERT_ERR_CUDA;
  // scalars only from here on
  ly->d.w_qkv = ly->d.w_o = ly->d.w_f1 = ly->d.w_f2 = nullptr;
  holder.p = nullptr;
  *out = ly;
  return IBERT_OK;
  });
}

// bytes of workspace one encoder-layer call needs for T tokens
static size_t layer_workspace_bytes(int H, int F, int64_t T) {
  auto up256 = [](size_t v) { return (v + 255) & ~size_t(255); };
  return up256((size_t)T * 3 * H) + up256((size_t)T * H) + up256((size_t)T * H * 4) + up256((size_t)T * H) +
         up256((size_t)T * F);
}

// cu_seqlens != nullptr: packed batch of `total` rows (sequence b = rows cu_seqlens[b] .. cu_seqlens[b+1]-1,
// at most L each); otherwise B padded sequences of L rows
static int encoder_layer_common(ibert_ctx* ctx, const ibert_layer* ly, const int8_t* x, int B, int L,
                                const int32_t* lens, int8_t* out, double* S_ret, const int32_t* cu_seqlens = nullptr,
                                int64_t total = 0) {
  if (!ctx || !ly || ly->ctx != ctx || B < 0) return IBERT_ERR_ARG;
  if (L < 1 || L > 512) return IBERT_ERR_SHAPE;
  const int H = ly->d.H, F = ly->d.F;
  if (cu_seqlens && (total < 0 || total > (int64_t)B * L || total >= (int64_t(1) << 31) - 256)) return IBERT_ERR_SHAPE;
  const int64_t T = cu_seqlens ? total : (int64_t)B * L;
  if (T > 0 && (!x || !out)) return IBERT_ERR_ARG;
  if (!aligned16(x) || !aligned16(out)) return IBERT_ERR_ALIGN;
  if (S_ret) *S_ret = ly->d.S_out;
  if (T == 0) return IBERT_OK;
  DeviceGuard guard(ctx->device);
  // workspace: qkv [T,3H] i8 | ctx [T,H] i8 | r [T,H] i32 (both residual sums) | h1 [T,H] i8 | g [T,F] i8
  auto up256 = [](size_t v) { return (v + 255) & ~size_t(255); };
  const size_t o_qkv = 0;
  const size_t o_ctx = o_qkv + up256((size_t)T * 3 * H);
  const size_t o_r = o_ctx + up256((size_t)T * H);
  const size_t o_h1 = o_r + up256((size_t)T * H * 4);
  const size_t o_g = o_h1 + up256((size_t)T * H);
  const size_t need = o_g + up256((size_t)T * F);
  if (int rcw = ensure_workspace(ctx, need)) return rcw;
  char* ws = static_cast<char*>(ctx->ws);
  int8_t* qkv = (int8_t*)(ws + o_qkv);
  int8_t* cx = (int8_t*)(ws + o_ctx);
  int16_t* r = (int16_t*)(ws + o_r);             // Q16 residual sums as int16 (two-kernel path only)
  int8_t* h1 = (int8_t*)(ws + o_h1);
  int8_t* g = (int8_t*)(ws + o_g);

  GemmEpilogue e{};
  int rc;
  e.kind = EPI_INT8; e.d_b = ly->b_qkv; e.d_c = ly->c_qkv; e.d_bias = ly->bias_qkv; e.fast = ly->fast_qkv;
  // Q | K | V between the two kernels: transposed ([3H][T]) where both sides take it -- a thread of the GEMM
  // holds one channel of 32 tokens, which are contiguous bytes of that layout
  const bool qkv_t = ctx->qkv_layout_mode != 1 && !cu_seqlens && ly->fast_qkv == 1 &&
                     attention_takes_transposed(B, L, ly->attn);
  e.out_transposed = qkv_t;
  { ProfileScope ps(ctx, IBERT_K_GEMM_QKV); rc = launch_gemm_i8(ctx, x, ly->w_qkv, T, 3 * H, H, e, qkv); }
  e.out_transposed = false;
  if (rc) return rc;
  { ProfileScope ps(ctx, IBERT_K_ATTENTION); rc = launch_attention(ctx, qkv, B, L, H, ly->d.heads, ly->attn, lens, cx, cu_seqlens, T, qkv_t); }
  if (rc) return rc;
  // output projection + residual + LayerNorm: one kernel when shapes and constants allow it
  e.kind = EPI_Q16; e.d_b = ly->b_o; e.d_c = ly->c_o; e.d_bias = ly->bias_o; e.fast = ly->fast_o;
  // the cluster kernel pays off once its 128-token tiles keep at least half of the SMs busy; below
  // that the two kernels, which spread a small problem over more CTAs, are faster
  const bool fuse = gemm_ln_profitable(ctx, T, H);
  if (fuse && gemm_ln_supported(H, H, e, ly->ln1)) {
    ProfileScope ps(ctx, IBERT_K_GEMM_LN);
    rc = launch_gemm_ln_i8(ctx, cx, ly->w_o, T, H, H, e, x, ly->ln1, ly->ln1_b, ly->ln1_B, h1);
  } else {
    e.kind = EPI_Q16H;
    { ProfileScope ps(ctx, IBERT_K_GEMM_Q16); rc = launch_gemm_i8(ctx, cx, ly->w_o, T, H, H, e, r); }
    if (rc) return rc;
    { ProfileScope ps(ctx, IBERT_K_LAYERNORM); rc = launch_layernorm_i16(ctx, r, x, T, ly->ln1, ly->ln1_b, ly->ln1_B, h1); }
  }
  if (rc) return rc;
  GemmEpilogue e2{};
  e2.kind = EPI_Q16; e2.d_b = ly->b_f2; e2.d_c = ly->c_f2; e2.d_bias = ly->bias_f2; e2.fast = ly->fast_f2;
  const bool fuse2 = fuse && gemm_ln_supported(H, F, e2, ly->ln2);
  // the FFN1 result between its GEMM and the cluster kernel: transposed ([F][T]) where both sides take it
  // (the table epilogue of a CTA-pair sized problem on one side, the fused kernel on the other)
  // (a tensor that no longer fits L2 comes back from HBM, where the fused kernel's channel-major tiles --
  // 128 rows of 128 bytes, T bytes apart -- read slower than token-major ones: T = 32768, F = 4096, 128 MB,
  // loses 1.5 % of the step)
  const bool g_pays = T >= 4096 && (int64_t)T * F <= ctx->l2_bytes / 2;
  const bool g_t = fuse2 && ctx->qkv_layout_mode != 1 && (g_pays || ctx->qkv_layout_mode == 2) && ly->gelu_table &&
                   ctx->gelu_table_mode == 0 && ly->fast_f1 != 0 && ly->gelu.fast != 0 &&
                   gemm_gelu_takes_transposed(ctx, T, F);
  e.kind = EPI_GELU; e.d_b = ly->b_f1; e.d_c = ly->c_f1; e.d_bias = ly->bias_f1; e.gelu = ly->gelu; e.fast = ly->fast_f1; e.gelu_table = ly->gelu_table;
  e.out_transposed = g_t;
  { ProfileScope ps(ctx, IBERT_K_GEMM_GELU); rc = launch_gemm_i8(ctx, h1, ly->w_f1, T, F, H, e, g); }
  e.out_transposed = false;
  if (rc) return rc;
  e.kind = EPI_Q16; e.d_b = ly->b_f2; e.d_c = ly->c_f2; e.d_bias = ly->bias_f2; e.fast = ly->fast_f2;
  if (fuse2) {
    ProfileScope ps(ctx, F > 2048 ? IBERT_K_GEMM_LN_WIDE : IBERT_K_GEMM_LN);
    return launch_gemm_ln_i8(ctx, g, ly->w_f2, T, H, F, e, h1, ly->ln2, ly->ln2_b, ly->ln2_B, out, g_t);
  }
  e.kind = EPI_Q16H;
  { ProfileScope ps(ctx, IBERT_K_GEMM_Q16_WIDE); rc = launch_gemm_i8(ctx, g, ly->w_f2, T, H, F, e, r); }
  if (rc) return rc;
  { ProfileScope ps(ctx, IBERT_K_LAYERNORM); rc = launch_layernorm_i16(ctx, r, h1, T, ly->ln2, ly->ln2_b, ly->ln2_B, out); }
  return rc;
}

int ibert_encoder_layer(ibert_ctx* ctx, const ibert_layer* ly, const int8_t* x, int B, int L,
                        int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  return encoder_layer_common(ctx, ly, x, B, L, nullptr, out, S_ret);
  });
}

int ibert_encoder_layer_masked(ibert_ctx* ctx, const ibert_layer* ly, const int8_t* x, int B, int L,
                               const int32_t* lens, int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  if (B > 0 && !lens) return IBERT_ERR_ARG;
  return encoder_layer_common(ctx, ly, x, B, L, lens, out, S_ret);
  });
}

int ibert_encoder_layer_packed(ibert_ctx* ctx, const ibert_layer* ly, const int8_t* x, const int32_t* cu_seqlens,
                               int B, int max_len, int64_t total_tokens, int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  if (B > 0 && !cu_seqlens) return IBERT_ERR_ARG;
  if (B == 0 && total_tokens != 0) return IBERT_ERR_ARG;
  return encoder_layer_common(ctx, ly, x, B, max_len, nullptr, out, S_ret, cu_seqlens, total_tokens);
  });
}

int ibert_attention_packed_i8(ibert_ctx* ctx, const int8_t* qkv, const int32_t* cu_seqlens, int B, int max_len,
                              int64_t total_tokens, int H, int heads, double S_q, double S_k, double S_v,
                              double S_ctx, int p_max, int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  if (!ctx || B < 0 || (B > 0 && !cu_seqlens)) return IBERT_ERR_ARG;
  if (heads < 1 || H != heads * 64 || max_len < 1 || max_len > 512) return IBERT_ERR_SHAPE;
  if (total_tokens < 0 || total_tokens > (int64_t)B * max_len || total_tokens >= (int64_t(1) << 31) - 256) return IBERT_ERR_SHAPE;
  if (total_tokens > 0 && (!qkv || !out)) return IBERT_ERR_ARG;
  if (!aligned16(qkv) || !aligned16(out)) return IBERT_ERR_ALIGN;
  AttnConsts k{};
  int rc = make_attn_consts(S_q, S_k, S_v, S_ctx, p_max, &k);
  if (rc) return rc;
  if (S_ret) *S_ret = S_ctx;
  if (total_tokens == 0) return IBERT_OK;
  DeviceGuard guard(ctx->device);
  ProfileScope ps(ctx, IBERT_K_ATTENTION);
  return launch_attention(ctx, qkv, B, max_len, H, heads, k, nullptr, out, cu_seqlens, total_tokens);
  });
}

static int embedding_common(ibert_ctx* ctx, const int32_t* ids, int64_t T, int L, const int8_t* word, int64_t V,
                            double S_word, const int8_t* pos, int64_t P, double S_pos, const double* gamma,
                            const double* beta, int H, double S_out, int8_t* out, double* S_ret,
                            const int32_t* cu_seqlens, int B);

int ibert_embedding_i8(ibert_ctx* ctx, const int32_t* ids, int64_t T, int L, const int8_t* word, int64_t V,
                       double S_word, const int8_t* pos, int64_t P, double S_pos, const double* gamma,
                       const double* beta, int H, double S_out, int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  return embedding_common(ctx, ids, T, L, word, V, S_word, pos, P, S_pos, gamma, beta, H, S_out, out, S_ret, nullptr, 0);
  });
}

int ibert_embedding_packed_i8(ibert_ctx* ctx, const int32_t* ids, const int32_t* cu_seqlens, int B, int max_len,
                              int64_t total_tokens, const int8_t* word, int64_t V, double S_word, const int8_t* pos,
                              int64_t P, double S_pos, const double* gamma, const double* beta, int H, double S_out,
                              int8_t* out, double* S_ret) {
  return guarded([&]() -> int {
  if (B < 0 || (B > 0 && !cu_seqlens) || (B == 0 && total_tokens != 0)) return IBERT_ERR_ARG;
  if (total_tokens > (int64_t)B * max_len) return IBERT_ERR_SHAPE;
  return embedding_common(ctx, ids, total_tokens, max_len, word, V, S_word, pos, P, S_pos, gamma, beta, H, S_out, out,
                          S_ret, cu_seqlens, B);
  });
}

static int embedding_common(ibert_ctx* ctx, const int32_t* ids, int64_t T, int L, const int8_t* word, int64_t V,
                            double S_word, const int8_t* pos, int64_t P, double S_pos, const double* gamma,
                            const double* beta, int H, double S_out, int8_t* out, double* S_ret,
                            const int32_t* cu_seqlens, int B) {
  if (!ctx || T < 0 || !gamma || !beta || !word || !pos) return IBERT_ERR_ARG;
  if (L < 1 || H < 1 || H > 2047 || H % 16 != 0 || V < 1 || P < L) return IBERT_ERR_SHAPE;
  if (T > 0 && (!ids || !out)) return IBERT_ERR_ARG;
  if (!aligned16(word) || !aligned16(pos) || !aligned16(out)) return IBERT_ERR_ALIGN;
  if (!good_scale(S_word) || !good_scale(S_pos) || !good_scale(S_out)) return IBERT_ERR_SCALE_RANGE;
  LnConsts k{};
  k.C = H;
  k.has_res = 1;
  int rc = make_ln_residual(S_pos, S_word, &k);
  if (rc) return rc;
  std::vector<int32_t> b_i;
  std::vector<int64_t> B_i;
  rc = make_ln_tables(gamma, beta, H, S_out, &k, &b_i, &B_i);
  if (rc) return rc;
  if (S_ret) *S_ret = S_out;
  if (T == 0) return IBERT_OK;
  DeviceGuard guard(ctx->device);
  if ((rc = trim_tables(ctx))) return rc;
  void *d_b = nullptr, *d_B = nullptr;
  if ((rc = cached_upload(ctx, b_i.data(), b_i.size() * sizeof(int32_t), 11, &d_b))) return rc;
  if ((rc = cached_upload(ctx, B_i.data(), B_i.size() * sizeof(int64_t), 12, &d_B))) return rc;
  // gathered rows: q int32 [T, H] (word row) | r int8 [T, H] (position row)
  const size_t q_bytes = ((size_t)T * H * 4 + 255) & ~size_t(255);
  if ((rc = ensure_workspace(ctx, q_bytes + (size_t)T * H + 256))) return rc;
  int32_t* q = static_cast<int32_t*>(ctx->ws);
  int8_t* r = reinterpret_cast<int8_t*>(static_cast<char*>(ctx->ws) + q_bytes);
  if ((rc = launch_embed_gather(ctx, ids, T, L, word, V, pos, H, q, r, cu_seqlens, B))) return rc;
  ProfileScope ps(ctx, IBERT_K_LAYERNORM);
  return launch_layernorm(ctx, q, r, T, k, (const int32_t*)d_b, (const int64_t*)d_B, out);
}

static int classifier_common(ibert_ctx* ctx, const int8_t* x, int B, int L, int H, double S_x, const int8_t* w,
                             const double* S_w, const int32_t* bias, int N, int32_t* logits, double* S_ret,
                             const int32_t* cu_seqlens);

int ibert_classifier_i8(ibert_ctx* ctx, const int8_t* x, int B, int L, int H, double S_x, const int8_t* w,
                        const double* S_w, const int32_t* bias, int N, int32_t* logits, double* S_ret) {
  return guarded([&]() -> int {
  return classifier_common(ctx, x, B, L, H, S_x, w, S_w, bias, N, logits, S_ret, nullptr);
  });
}

int ibert_classifier_packed_i8(ibert_ctx* ctx, const int8_t* x, const int32_t* cu_seqlens, int B, int H, double S_x,
                               const int8_t* w, const double* S_w, const int32_t* bias, int N, int32_t* logits,
                               double* S_ret) {
  return guarded([&]() -> int {
  if (B > 0 && !cu_seqlens) return IBERT_ERR_ARG;
  return classifier_common(ctx, x, B, 1, H, S_x, w, S_w, bias, N, logits, S_ret, cu_seqlens);
  });
}

static int classifier_common(ibert_ctx* ctx, const int8_t* x, int B, int L, int H, double S_x, const int8_t* w,
                             const double* S_w, const int32_t* bias, int N, int32_t* logits, double* S_ret,
                             const int32_t* cu_seqlens) {
  if (!ctx || B < 0 || !S_w || !w) return IBERT_ERR_ARG;
  if (L < 1 || H < 1 || H % 16 != 0 || N < 1 || N % 4 != 0) return IBERT_ERR_SHAPE;
  if ((int64_t)H * 127 * 127 >= (int64_t(1) << 31)) return IBERT_ERR_SHAPE;
  if (B > 0 && (!x || !logits)) return IBERT_ERR_ARG;
  if (!aligned16(x) || !aligned16(w) || !aligned16(logits) || (bias && !aligned16(bias))) return IBERT_ERR_ALIGN;
  if (!good_scale(S_x)) return IBERT_ERR_SCALE_RANGE;
  for (int n = 0; n < N; ++n)
    if (!good_scale(S_w[n])) return IBERT_ERR_SCALE_RANGE;
  if (S_ret) for (int n = 0; n < N; ++n) S_ret[n] = S_x * S_w[n];
  if (B == 0) return IBERT_OK;
  DeviceGuard guard(ctx->device);
  int rc = ensure_workspace(ctx, (size_t)B * H + 256);
  if (rc) return rc;
  int8_t* first = static_cast<int8_t*>(ctx->ws);
  // first token of every sequence: B rows of H bytes, L*H bytes apart (packed: row cu_seqlens[b])
  if (cu_seqlens) {
    if ((rc = launch_gather_first_rows(ctx, x, cu_seqlens, B, H, first))) return rc;
  } else if (cudaMemcpy2DAsync(first, (size_t)H, x, (size_t)L * H, (size_t)H, (size_t)B, cudaMemcpyDeviceToDevice,
                               ctx->stream) != cudaSuccess) { cudaGetLastError(); return IBERT_ERR_CUDA; }
  GemmEpilogue epi{};
  epi.kind = EPI_RAW;
  epi.d_bias = bias;
  ProfileScope ps(ctx, gemm_class(EPI_RAW, H));
  return launch_gemm_i8(ctx, first, w, B, N, H, epi, logits);
}

// --------------------------------------------------------------------------- captured forward pass
// A stack of encoder layers for fixed shapes and fixed buffers, captured once into a CUDA graph:
// small batches are bound by launch overhead (60 launches per 12-layer pass), which a graph replay
// removes.  The graph owns its workspace and its ping-pong activation buffers.
struct ibert_graph {
  ibert_ctx* ctx = nullptr;
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;
  void* ws = nullptr;
  size_t ws_bytes = 0;
  int8_t* bufs[2] = {nullptr, nullptr};
};

static void graph_free(ibert_graph* g) {
  if (g->exec) cudaGraphExecDestroy(g->exec);
  if (g->graph) cudaGraphDestroy(g->graph);
  if (g->ws) cudaFree(g->ws);
  for (int i = 0; i < 2; ++i) if (g->bufs[i]) cudaFree(g->bufs[i]);
  delete g;
}

int ibert_encoder_graph_create(ibert_ctx* ctx, const ibert_layer* const* layers, int n_layers, const int8_t* x,
                               int B, int L, const int32_t* lens, int8_t* out, ibert_graph** out_graph) {
  return guarded([&]() -> int {
  if (!ctx || !layers || n_layers < 1 || !out_graph || B < 1 || !x || !out) return IBERT_ERR_ARG;
  *out_graph = nullptr;
  if (L < 1 || L > 512) return IBERT_ERR_SHAPE;
  if (ctx->profiling) return IBERT_ERR_ARG;                 // events cannot be recorded into the capture
  if (ctx->stream == nullptr) return IBERT_ERR_ARG;         // the default stream cannot be captured
  const int H = layers[0] ? layers[0]->d.H : 0;
  size_t need = 0;
  for (int i = 0; i < n_layers; ++i) {
    if (!layers[i] || layers[i]->ctx != ctx || layers[i]->d.H != H) return IBERT_ERR_ARG;
    need = std::max(need, layer_workspace_bytes(H, layers[i]->d.F, (int64_t)B * L));
  }
  if (!aligned16(x) || !aligned16(out)) return IBERT_ERR_ALIGN;
  DeviceGuard guard(ctx->device);
  ibert_graph* g = new (std::nothrow) ibert_graph();
  if (!g) return IBERT_ERR_NOMEM;
  g->ctx = ctx;
  const size_t act = (size_t)B * L * H;
  if (cudaMalloc(&g->ws, need) != cudaSuccess ||
      (n_layers > 1 && (cudaMalloc((void**)&g->bufs[0], act) != cudaSuccess ||
                        cudaMalloc((void**)&g->bufs[1], act) != cudaSuccess))) {
    cudaGetLastError();
    graph_free(g);
    return IBERT_ERR_NOMEM;
  }
  g->ws_bytes = need;
  // the layers run against the graph's own workspace, once eagerly (function attributes, cached
  // launch parameters, argument checks) and once under capture
  void* saved_ws = ctx->ws;
  const size_t saved_bytes = ctx->ws_bytes;
  ctx->ws = g->ws;
  ctx->ws_bytes = g->ws_bytes;
  auto run = [&]() {
    for (int i = 0; i < n_layers; ++i) {
      const int8_t* in = i == 0 ? x : g->bufs[(i - 1) & 1];
      int8_t* o = i == n_layers - 1 ? out : g->bufs[i & 1];
      if (int rc = encoder_layer_common(ctx, layers[i], in, B, L, lens, o, nullptr)) return rc;
    }
    return (int)IBERT_OK;
  };
  int rc = run();
  if (rc == IBERT_OK && cudaStreamSynchronize(ctx->stream) != cudaSuccess) rc = IBERT_ERR_CUDA;
  if (rc == IBERT_OK) {
    if (cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) rc = IBERT_ERR_CUDA;
    else {
      rc = run();
      cudaGraph_t captured = nullptr;
      if (cudaStreamEndCapture(ctx->stream, &captured) != cudaSuccess) { cudaGetLastError(); if (rc == IBERT_OK) rc = IBERT_ERR_CUDA; }
      g->graph = captured;
      if (rc == IBERT_OK && cudaGraphInstantiate(&g->exec, g->graph, 0) != cudaSuccess) { cudaGetLastError(); rc = IBERT_ERR_CUDA; }
    }
  }
  ctx->ws = saved_ws;
  ctx->ws_bytes = saved_bytes;
  if (rc != IBERT_OK) { graph_free(g); return rc; }
  *out_graph = g;
  return IBERT_OK;
  });
}

int ibert_encoder_graph_launch(ibert_ctx* ctx, ibert_graph* g) {
  return guarded([&]() -> int {
  if (!ctx || !g || g->ctx != ctx || !g->exec) return IBERT_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (cudaGraphLaunch(g->exec, ctx->stream) != cudaSuccess) { cudaGetLastError(); return IBERT_ERR_CUDA; }
  return IBERT_OK;
  });
}

int ibert_encoder_graph_destroy(ibert_graph* g) {
  return guarded([&]() -> int {
  if (!g) return IBERT_ERR_ARG;
  DeviceGuard guard(g->ctx->device);
  cudaStreamSynchronize(g->ctx->stream);
  graph_free(g);
  return IBERT_OK;
  });
}

int ibert_selftest_exp_division(double S, int32_t* q_ln2_out) {
  return guarded([&]() -> int {
  ExpConsts k;
  int rc = make_exp_consts(S, 255, &k);
  if (rc) return rc;
  if (q_ln2_out) *q_ln2_out = (int32_t)k.q_ln2;
  for (uint32_t d = 0; d <= k.d_max; ++d) {
    const uint64_t wide = (uint64_t)(uint32_t)(d << k.div_pre) * (uint64_t)k.div_m;
    const uint32_t z = (uint32_t)(wide >> 32) >> k.div_post;
    if (z != d / k.q_ln2) return IBERT_ERR_VALUE_RANGE;
  }
  if (k.wide_post >= 0) {            // the unclamped form used on attention scores: every d < 2^21
    for (uint32_t d = 0; d < (1u << 21); ++d) {
      const uint32_t z = (uint32_t)(((uint64_t)d * (uint64_t)k.wide_m) >> 32) >> k.wide_post;
      if (z != d / k.q_ln2) return IBERT_ERR_VALUE_RANGE;
    }
  }
  return IBERT_OK;
  });
}

int ibert_selftest_wait_timeout(ibert_ctx* ctx, int64_t limit_us) {
  return guarded([&]() -> int {
  if (!ctx || limit_us < 1 || limit_us > 100000) return IBERT_ERR_ARG;
  DeviceGuard guard(ctx->device);
  return launch_wait_timeout(ctx, (uint64_t)limit_us * 1000ull);
  });
}

int ibert_profile_begin(ibert_ctx* ctx) {
  return guarded([&]() -> int {
  if (!ctx) return IBERT_ERR_ARG;
  ctx->ev_class.clear();
  ctx->profiling = true;
  return IBERT_OK;
  });
}

int ibert_profile_end(ibert_ctx* ctx, float* ms, int32_t* launches) {
  return guarded([&]() -> int {
  if (!ctx || !ms || !launches) return IBERT_ERR_ARG;
  DeviceGuard guard(ctx->device);
  ctx->profiling = false;
  for (int i = 0; i < IBERT_NUM_KERNEL_CLASSES; ++i) { ms[i] = 0.f; launches[i] = 0; }
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return IBERT_ERR_CUDA;
  for (size_t i = 0; i < ctx->ev_class.size(); ++i) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, ctx->ev_pool[2 * i], ctx->ev_pool[2 * i + 1]) != cudaSuccess) {
      cudaGetLastError();
      continue;
    }
    ms[ctx->ev_class[i]] += t;
    launches[ctx->ev_class[i]] += 1;
  }
  ctx->ev_class.clear();
  return IBERT_OK;
  });
}

}  // extern "C"
