// Status strings, error bookkeeping and the host-only position-layout helpers
// (AMA, UPL, <o> and step-block PIDs; paper Sec. 2.1.2 and Sec. 2.2).
#include <atomic>

#include "common.cuh"

namespace ms {

static std::atomic<unsigned int> g_wait_limit_us{4000000u};

unsigned int wait_limit_us() { return g_wait_limit_us.load(std::memory_order_relaxed); }

static thread_local int32_t g_last_cuda_error = 0;

void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = static_cast<int32_t>(e); }

int32_t sm_count() {
  static int32_t cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    cached[dev] = n;
  }
  return cached[dev];
}

}  // namespace ms

extern "C" {

int32_t memosight_version(void) { return 100; }

const char* memosight_status_string(int32_t status) {
  switch (status) {
    case MS_OK: return "ok";
    case MS_ERR_INVALID_ARG: return "invalid argument";
    case MS_ERR_UNSUPPORTED_SHAPE: return "shape outside the supported limits";
    case MS_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case MS_ERR_ALIGNMENT: return "pointer or stride not 16-byte aligned";
    case MS_ERR_CUDA: return "CUDA call failed";
    case MS_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    default: return "unknown status";
  }
}

int32_t memosight_last_cuda_error(void) { return ms::g_last_cuda_error; }

uint32_t memosight_debug_set_wait_limit_us(uint32_t limit_us) {
  if (limit_us == 0) return ms::g_wait_limit_us.load(std::memory_order_relaxed);
  return ms::g_wait_limit_us.exchange(limit_us, std::memory_order_relaxed);
}

// l = ceil(n / c)  (Sec. 2.1.2, Adaptive Memory Allocation)
int32_t memosight_ama(int32_t n, int32_t c) {
  if (n < 0 || c < 1) return MS_ERR_INVALID_ARG;
  return static_cast<int32_t>((static_cast<int64_t>(n) + c - 1) / c);
}

// Centre PID of each of the l groups (Sec. 2.1.2, Uniform Position Layout).
int32_t memosight_upl_pids(int32_t rho_first, int32_t n, int32_t c, uint32_t flags,
                           int32_t* pid_out, int32_t cap) {
  const int32_t l = memosight_ama(n, c);
  if (l < 0) return l;
  if (l > 0 && (pid_out == nullptr || cap < l)) return MS_ERR_INVALID_ARG;
  if (flags & ~(MS_POS_HALF_UNITS | MS_LAYOUT_MONOTONE)) return MS_ERR_INVALID_ARG;
  if (flags & MS_LAYOUT_MONOTONE) {   // "w/o UPL": fresh PIDs behind the step, one per memory token
    const int32_t unit = (flags & MS_POS_HALF_UNITS) ? 2 : 1;
    for (int32_t g = 0; g < l; ++g) pid_out[g] = unit * (rho_first + n + g);
    return l;
  }
  for (int32_t g = 0; g < l; ++g) {
    const int64_t first = static_cast<int64_t>(g) * c;               // offsets inside the step
    const int64_t last = (first + c < n ? first + c : n) - 1;
    const int64_t twice_centre = 2 * static_cast<int64_t>(rho_first) + first + last;
    pid_out[g] = static_cast<int32_t>((flags & MS_POS_HALF_UNITS) ? twice_centre
                                                                 : (twice_centre >> 1));
  }
  return l;
}

// Fixed budget of l memory tokens ("w/o AMA"): l groups cut as evenly as possible.
int32_t memosight_budget_pids(int32_t rho_first, int32_t n, int32_t l, int32_t* pid_out, int32_t cap) {
  if (n < 1 || l < 1 || pid_out == nullptr || cap < l) return MS_ERR_INVALID_ARG;
  for (int32_t g = 0; g < l; ++g) {
    int64_t first = static_cast<int64_t>(g) * n / l;
    int64_t last = static_cast<int64_t>(g + 1) * n / l - 1;
    if (last < first) last = first;               // empty group: where it would start
    if (first > n - 1) first = n - 1;
    if (last > n - 1) last = n - 1;
    pid_out[g] = rho_first + static_cast<int32_t>((first + last) >> 1);
  }
  return l;
}

int32_t memosight_out_pid(int32_t rho_first, int32_t n) { return rho_first + n; }

// Candidates count up from p0; foresight token k sits k positions after the last
// regular token it can see (Sec. 2.1.1; Sec. 2.2).
int32_t memosight_step_pids(int32_t p0, int32_t n_c, int32_t d, const int32_t* anchor,
                            int32_t* pid_out) {
  if (n_c < 0 || d < 0 || (n_c + d > 0 && pid_out == nullptr)) return MS_ERR_INVALID_ARG;
  for (int32_t k = 0; k < d; ++k)
    if (anchor && (anchor[k] < 0 || anchor[k] > n_c)) return MS_ERR_INVALID_ARG;
  for (int32_t i = 0; i < n_c; ++i) pid_out[i] = p0 + i;
  for (int32_t k = 0; k < d; ++k) {
    const int32_t seen = anchor ? anchor[k] : n_c;
    pid_out[n_c + k] = p0 + seen + k;   // (p0 + seen - 1) + (k + 1)
  }
  return MS_OK;
}

}  // extern "C"
