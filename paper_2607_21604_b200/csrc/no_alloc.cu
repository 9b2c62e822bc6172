// Probe selection for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a serving loop whose
// memory pool is fixed at start-up, in a process that has handed all remaining device memory
// to another allocator, or under a policy that forbids allocation on the request path.
// akvs_op_select needs scratch (sort keys, selection flags, counters) that such a caller has
// nowhere to take from.  akvs_op_select_static is the same selection with that scratch held
// in a fixed array inside the library's own device image: loading the library reserves it on
// every GPU that loads it (about 0.3 MB) until the process exits, and no call allocates.
#include "common.cuh"

namespace {

constexpr int kMaxCtx = AKVS_STATIC_MAX_CTX;        // context tokens per request
constexpr int kMaxUnits = AKVS_STATIC_MAX_UNITS;
constexpr size_t kStatusBytes = 256;                 // status word + row counters, padded
constexpr size_t kKeysBytes = 2ull * kMaxCtx * sizeof(uint64_t);
constexpr size_t kFlagsBytes = 2ull * kMaxCtx;
constexpr size_t kScratchBytes = kStatusBytes + kKeysBytes + kFlagsBytes;

// The scratch itself.  In host code this name is only a handle for the runtime's symbol
// calls; the device address is obtained with cudaGetSymbolAddress, per device.
static __device__ __align__(256) unsigned char g_select_scratch[kScratchBytes];

// One resolved address per device ordinal.  Written without synchronisation: like the rest of
// the library's host state it relies on the convention that one host thread drives one device
// per process.  An address stays valid for the life of the process's context on that device;
// after a cudaDeviceReset the library must not be used any further (its module state is gone).
constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch on the current device; resolved on the first call per device.
int32_t scratch_address(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AKVS_ERR_CUDA;
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_select_scratch) != cudaSuccess || !p) return AKVS_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = reinterpret_cast<unsigned char*>(g_scratch_ptr[dev]);
  return AKVS_OK;
}

}  // namespace

extern "C" int32_t akvs_op_select_static(const float* d_k, const float* d_v, const int32_t* ctx_off_host,
                                         int32_t n_units, int32_t n_query, int32_t refresh_bp, akvs_probes* out,
                                         void* stream) {
  if (!d_k || !d_v || !ctx_off_host || !out || n_units < 0 || n_query < 0 || refresh_bp < 0 || refresh_bp > 10000)
    return AKVS_ERR_INVALID_ARG;
  if (!out->ctx_off || !out->probe_off || !out->sk_idx || !out->sv_idx || !out->w_k || !out->w_v || !out->rows)
    return AKVS_ERR_INVALID_ARG;
  if (n_units > kMaxUnits) return AKVS_ERR_TOO_LARGE;
  const int M = n_units;
  int32_t probe_off[kMaxUnits + 1];                  // on the stack: no host allocation either
  probe_off[0] = 0;
  for (int u = 0; u < M; ++u) {
    const int64_t n = (int64_t)ctx_off_host[u + 1] - ctx_off_host[u];
    if (n < 0) return AKVS_ERR_SHAPE;
    int64_t b = (n * refresh_bp + 9999) / 10000;
    b = b > n ? n : b;
    probe_off[u + 1] = probe_off[u] + (int32_t)b;
  }
  const int N = ctx_off_host[M];
  if (ctx_off_host[0] != 0 || N < 0) return AKVS_ERR_SHAPE;
  if (N > kMaxCtx) return AKVS_ERR_TOO_LARGE;

  unsigned char* base = nullptr;
  AKVS_TRY(scratch_address(&base));
  int32_t* status = reinterpret_cast<int32_t*>(base);
  uint64_t* keys = reinterpret_cast<uint64_t*>(base + kStatusBytes);
  uint8_t* flags = base + kStatusBytes + kKeysBytes;

  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  // the array keeps the previous call's contents: the status word and counters must start at
  // zero; keys and flags are rewritten for all N tokens before they are read
  AKVS_CUDA(cudaMemsetAsync(status, 0, kStatusBytes, st));
  AKVS_CUDA(cudaMemcpyAsync(out->ctx_off, ctx_off_host, (M + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  AKVS_CUDA(cudaMemcpyAsync(out->probe_off, probe_off, (M + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  AKVS_TRY(launch_select(d_k, d_v, out->ctx_off, out->probe_off, M, N, n_query, out->sk_idx, out->sv_idx, out->w_k,
                         out->w_v, out->rows, keys, flags, status + 4, status, st));
  int32_t host[8] = {0};
  AKVS_CUDA(cudaMemcpyAsync(host, status, sizeof(host), cudaMemcpyDeviceToHost, st));
  AKVS_CUDA(cudaStreamSynchronize(st));
  if (host[0] != 0) return host[0];
  out->n_ctx = N;
  out->n_probe_rows = host[4];
  out->n_rows = host[5];
  return AKVS_OK;
}
