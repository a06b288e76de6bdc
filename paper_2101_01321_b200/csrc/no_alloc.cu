// ibert_layernorm_i_static: residual + i-LayerNorm for callers that must not allocate.
//
// The ordinary entry point keeps its per-channel constant tables (multipliers b_i, addends B_i)
// in device memory it obtains with cudaMalloc.  Some callers cannot do that: code inside a
// memory-pool or real-time section where the allocator is off limits, a host thread that may not
// block on the driver's allocation lock, or a process whose device memory is entirely managed by
// someone else.  This variant keeps the tables (and its status word) in one file-scope device
// array instead, so the call performs no device allocation of any kind -- only an asynchronous
// copy of the tables and the kernel launch.
#include <cstring>
#include <mutex>
#include <new>

#include "ibert_internal.h"

namespace {

constexpr int kMaxC = IBERT_STATIC_LN_MAX_C;
constexpr int kMaxDevices = 64;

// layout: [0, 256) status word | b_i: kMaxC int32 | B_i: kMaxC int64; every part starts on a
// 256-byte boundary (the kernels read the tables with 16-byte vector loads)
constexpr size_t round_up_256(size_t v) { return (v + 255) & ~size_t(255); }
constexpr size_t kOffB = 256;
constexpr size_t kOffBig = round_up_256(kOffB + sizeof(int32_t) * kMaxC);
constexpr size_t kScratchBytes = round_up_256(kOffBig + sizeof(int64_t) * kMaxC);
static_assert(kOffB % 16 == 0 && kOffBig % 16 == 0, "vector loads need 16-byte aligned tables");

// Held by every GPU that loads the library until the process exits (24,832 bytes).
static __device__ __align__(256) unsigned char g_ln_scratch[kScratchBytes];

// The symbol above is only a host-side stand-in here; kernels need its device address, which
// differs per device and is looked up once per device with that device current.
unsigned char* g_scratch_addr[kMaxDevices] = {};
int g_num_sms[kMaxDevices] = {};
std::mutex g_lookup_mutex;         // first calls from several host threads

int scratch_for_current_device(int device, unsigned char** out) {
  if (device < 0 || device >= kMaxDevices) return IBERT_ERR_ARG;
  std::lock_guard<std::mutex> lock(g_lookup_mutex);
  if (!g_scratch_addr[device]) {
    unsigned char* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_ln_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return IBERT_ERR_CUDA;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1) {
      cudaGetLastError();
      return IBERT_ERR_CUDA;
    }
    g_num_sms[device] = sms;
    g_scratch_addr[device] = p;
  }
  *out = g_scratch_addr[device];
  return IBERT_OK;
}

}  // namespace

extern "C" int ibert_layernorm_i_static(void* cuda_stream, const int32_t* q, double S, const int8_t* r, double S_r,
                                        const double* gamma, const double* beta, int64_t rows, int C,
                                        double S_out, int8_t* out, double* S_ret) {
  try {
    using namespace ibert;
    if (rows < 0 || !gamma || !beta) return IBERT_ERR_ARG;
    if (C < 1 || C > kMaxC || C > 2047) return IBERT_ERR_SHAPE;        // beyond the static tables
    if (rows > 0 && (!q || !out)) return IBERT_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(r)) & 15u)
      return IBERT_ERR_ALIGN;
    if (!(S > 0.0) || !(S_out > 0.0) || S != S || S_out != S_out || S > 1e300 || S_out > 1e300) return IBERT_ERR_SCALE_RANGE;
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

    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return IBERT_ERR_CUDA;
    unsigned char* scratch = nullptr;
    rc = scratch_for_current_device(device, &scratch);   // first call on a device: address lookup
    if (rc) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // The array keeps whatever the last call left.  The two tables are overwritten for all C
    // channels this call reads; the status word is not cleared here on purpose: it holds the first
    // device-side error since the last ibert_layernorm_i_static_status(), which clears it (the
    // array starts zeroed when the library is loaded).
    if (cudaMemcpyAsync(scratch + kOffB, b_i.data(), sizeof(int32_t) * C, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(scratch + kOffBig, B_i.data(), sizeof(int64_t) * C, cudaMemcpyHostToDevice, stream) != cudaSuccess)
      return IBERT_ERR_CUDA;
    // a context object on the stack: no device resources of its own
    ibert_ctx ctx;
    ctx.device = device;
    ctx.stream = stream;
    ctx.num_sms = g_num_sms[device];
    ctx.d_status = reinterpret_cast<int32_t*>(scratch);
    rc = launch_layernorm(&ctx, q, r, rows, k, reinterpret_cast<const int32_t*>(scratch + kOffB),
                          reinterpret_cast<const int64_t*>(scratch + kOffBig), out);
    if (rc == IBERT_OK && S_ret) *S_ret = S_out;
    return rc;
  } catch (const std::bad_alloc&) {
    return IBERT_ERR_NOMEM;
  } catch (...) {
    return IBERT_ERR_ARG;
  }
}

// Device-side status of the calls above on the current device since the last query: copies the
// status word out of the fixed array after synchronizing `cuda_stream`, clears it, and returns it
// (IBERT_OK, or IBERT_ERR_TIMEOUT when a bounded wait inside the kernel ran out).  Allocates nothing.
extern "C" int ibert_layernorm_i_static_status(void* cuda_stream) {
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess) return IBERT_ERR_CUDA;
  unsigned char* scratch = nullptr;
  if (int rc = scratch_for_current_device(device, &scratch)) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int32_t st = 0;
  if (cudaMemcpyAsync(&st, scratch, sizeof(st), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return IBERT_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return IBERT_ERR_CUDA;
  if (st != 0 && cudaMemsetAsync(scratch, 0, sizeof(st), stream) != cudaSuccess) return IBERT_ERR_CUDA;
  return st;
}
