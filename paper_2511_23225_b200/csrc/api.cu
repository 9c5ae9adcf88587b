// Library-wide helpers: status strings, error text, launch counter, workspace sizing.
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "common.cuh"

namespace {
std::atomic<uint64_t> g_launches{0};
thread_local char g_err[256] = "";
}  // namespace

namespace tweo_detail {

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

bool log_enabled() {
  static const bool on = [] {
    const char* v = getenv("TWEO_LOG");
    return v && *v && strcmp(v, "0") != 0;
  }();
  return on;
}

void log_call(const char* fmt, ...) {
  char line[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(line, sizeof line, fmt, ap);
  va_end(ap);
  fprintf(stderr, "[tweo] %s\n", line);
}

void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

tweo_status_t cuda_fail(cudaError_t e, const char* what) {
  snprintf(g_err, sizeof g_err, "%s: %s", what, cudaGetErrorString(e));
  return TWEO_ERR_CUDA;
}

tweo_status_t check_launch(const char* what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, what);
  return TWEO_OK;
}

size_t quantize_workspace_bytes();
size_t block_output_workspace_bytes();
size_t absmax_workspace_bytes();
// Blocks per tensor of the loss kernel; also fixes the workspace size.
int loss_blocks_per_tensor(int64_t n, int L);

}  // namespace tweo_detail

extern "C" {

const char* tweo_status_string(tweo_status_t s) {
  switch (s) {
    case TWEO_OK: return "ok";
    case TWEO_ERR_INVALID_ARG: return "invalid argument";
    case TWEO_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case TWEO_ERR_ALIGNMENT: return "pointer or row pitch not 16-byte aligned";
    case TWEO_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case TWEO_ERR_CUDA: return "CUDA call failed";
    case TWEO_ERR_TIMEOUT: return "a bounded device-side wait expired";
    default: return "unknown status";
  }
}

const char* tweo_last_cuda_error(void) { return g_err; }

int32_t tweo_version(void) { return 301; }

uint64_t tweo_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

size_t tweo_workspace_bytes(int32_t op, int64_t M, int64_t N, int64_t K) {
  const size_t sms = (size_t)tweo_detail::sm_count();
  const size_t stream_k_bytes = 12288 + sms * 256 * 1024;  // flags, ticket counters, 256 KB of parked fp32 sums per SM
  switch (op) {
    case TWEO_OP_QUANTIZE:
      return tweo_detail::quantize_workspace_bytes();  // optional: selects the batched form of the cast
    case TWEO_OP_LOSS: {
      int L = (int)(N < 1 ? 1 : N);
      return 256 + sizeof(double) * (size_t)L * (size_t)tweo_detail::loss_blocks_per_tensor(M, L);
    }
    case TWEO_OP_LINEAR_FWD:
    case TWEO_OP_LINEAR_DGRAD:
    case TWEO_OP_LINEAR_WGRAD:
      // optional: lets the GEMM split tiles along the contraction (parked fp32 accumulators + flags)
      return stream_k_bytes;
    case TWEO_OP_ABSMAX:
      return tweo_detail::absmax_workspace_bytes();
    case TWEO_OP_BLOCK_OUTPUT:
      return tweo_detail::block_output_workspace_bytes();
    case TWEO_OP_W8A8: {
      // scalars + codes of the activations (a bf16 input is cast inside) + the GEMM's stream-K area
      size_t codes = (size_t)(M < 0 ? 0 : M) * (size_t)(K < 0 ? 0 : K);
      codes = (codes + 255) & ~(size_t)255;
      return 256 + codes + stream_k_bytes;
    }
    default:
      return 0;
  }
}

tweo_status_t tweo_workspace_init(void* ws, size_t ws_bytes, void* stream) {
  if (ws_bytes == 0) return TWEO_OK;
  if (!ws) return TWEO_ERR_INVALID_ARG;
  TWEO_CUDA_TRY(cudaMemsetAsync(ws, 0, ws_bytes, (cudaStream_t)stream));
  return TWEO_OK;
}

tweo_status_t tweo_read_device_status(void* stream) {
  return tweo_detail::read_and_clear_device_status((cudaStream_t)stream);
}

}  // extern "C"
