// "Last block done" counters.
//
// Several kernels of the library end with a small serial tail that needs the work of every
// thread block of the same launch: the log-sum-exp merge of an attention unit that was cut
// across blocks, the per-sequence prefix match of the greedy accept, the new cache lengths of
// a compaction.  Instead of a second launch, the block that finishes last does the tail; it
// knows it is last from one atomicAdd on a counter that started at zero.  No block ever waits
// for another.
//
// The counters cannot live in caller memory, which may hold anything when the library first
// sees it.  They live in a fixed array inside the library image (zero when the module loads),
// handed out in banks: the first call that names a key -- the address of the buffer the tail
// writes, which overlapping calls must not share anyway -- gets the next free bank on the
// current device and keeps it.  Every user puts its counters back to zero before its kernel
// ends, so a bank is zero between launches whatever happens to the caller's buffers.  When all
// banks are taken the callers fall back to their two-launch form.
#include <mutex>

#include "common.cuh"

namespace ms {
namespace {

constexpr int kDoneBanks = 128;   // x 2048 counters x 4 bytes = 1 MB per GPU that loads the library
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned int g_done_words[kDoneBanks * kDoneBankWords];

struct DeviceBanks {
  unsigned int* base = nullptr;
  int used = 0;
  const void* key[kDoneBanks];
};

std::mutex g_mu;
DeviceBanks g_banks[kMaxDevices];
int g_bank_limit = kDoneBanks;      // memosight_debug_set_bank_limit

}  // namespace

unsigned int* done_bank(const void* key) {
  int dev = 0;
  if (!key || cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_mu);
  DeviceBanks& d = g_banks[dev];
  if (!d.base) {
    // in host code the array's name is only a handle: ask the runtime for its device address
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_done_words) != cudaSuccess || !p) {
      (void)cudaGetLastError();
      return nullptr;
    }
    d.base = static_cast<unsigned int*>(p);
  }
  const int limit = g_bank_limit < kDoneBanks ? g_bank_limit : kDoneBanks;
  for (int i = (d.used < limit ? d.used : limit) - 1; i >= 0; --i)
    if (d.key[i] == key) return d.base + static_cast<size_t>(i) * kDoneBankWords;
  if (d.used >= limit) return nullptr;
  d.key[d.used] = key;
  return d.base + static_cast<size_t>(d.used++) * kDoneBankWords;
}

int32_t done_bank_clear(const void* key, cudaStream_t st) {
  unsigned int* bank = done_bank(key);
  if (!bank) return MS_OK;
  MS_CUDA_TRY(cudaMemsetAsync(bank, 0, sizeof(unsigned int) * kDoneBankWords, st));
  return MS_OK;
}

}  // namespace ms

extern "C" int32_t memosight_debug_set_bank_limit(int32_t n_banks) {
  std::lock_guard<std::mutex> lock(ms::g_mu);
  const int32_t prev = ms::g_bank_limit;
  if (n_banks >= 0) ms::g_bank_limit = n_banks;
  return prev;
}
