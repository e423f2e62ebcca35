// Acceptance-only entry point that never allocates.
//
// sled_accept_rows marshals its host-side request description (row offsets, draft ids,
// Philox counter words, per-request row pointers) into a small device block that it
// obtains from cudaMalloc on every call.  Some callers must not do that: code running
// inside a serving process whose device memory is entirely owned by another allocator
// (a framework's caching pool sized to the whole GPU), code on a latency path where an
// allocation would synchronise the device, and code that is not allowed to touch the
// allocator between two fixed points of its schedule.  For them the same kernel is
// offered with that block placed in a fixed array that is part of the library image.
#include <cstdio>
#include <cstring>

#include "../../include/sled.h"
#include "kernels.h"

namespace {

// Layout of the block, sized for the stated maxima.  Every GPU that loads the library
// holds this array (a little over 68 KB; under 69 KB, checked below) until the process exits.
constexpr int kMaxReqs = SLED_STATIC_MAX_REQS;
constexpr int kMaxRows = SLED_STATIC_MAX_ROWS;
struct alignas(256) StaticBlock {
  int32_t ids[kMaxRows];          // fed token per row (drafts at rows 1.. of a request)
  int32_t cu[kMaxReqs + 1];       // first row of each request
  uint32_t lo[kMaxReqs];          // context id, low / high word
  uint32_t hi[kMaxReqs];
  int32_t pos0[kMaxReqs];         // index of the pending token
  const void* qptr[kMaxReqs];     // device address of each request's draft rows
  int32_t results[3 * kMaxReqs];  // n_accepted, next_token, status
};

static_assert(sizeof(StaticBlock) < 69 * 1024, "the size stated in sled.h");

// In host code this name only stands for the symbol; it is not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticBlock)];

constexpr int kMaxDevices = 64;
StaticBlock* g_block_of_device[kMaxDevices] = {};  // filled once per device by the first call on it

// Device address of the array on the current device (asked for once per device).
int block_address(StaticBlock** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SLED_ERR_NO_DEVICE;
  if (!g_block_of_device[dev]) {
    void* p = nullptr;
    cudaError_t err = cudaGetSymbolAddress(&p, g_static_scratch);
    if (err != cudaSuccess || !p) {
      std::fprintf(stderr, "sled: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(err));
      return SLED_ERR_DEVICE;
    }
    g_block_of_device[dev] = static_cast<StaticBlock*>(p);
  }
  *out = g_block_of_device[dev];
  return SLED_OK;
}

}  // namespace

extern "C" int sled_accept_rows_static(const float* logits, const int32_t* cu_rows, const int32_t* drafts,
                                       const float* q_rows, const uint64_t* ctx_ids, const int64_t* pos0,
                                       int32_t n_reqs, int32_t vocab, float temperature, int32_t greedy,
                                       uint64_t seed, sled_result* results, void* stream) {
  if (!logits || !cu_rows || !ctx_ids || !pos0 || !results || n_reqs <= 0 || vocab <= 0 || !(temperature > 0.f))
    return SLED_ERR_ARG;
  if (n_reqs > kMaxReqs) {
    std::fprintf(stderr, "sled_accept_rows_static: %d requests exceed the fixed maximum of %d\n", n_reqs, kMaxReqs);
    return SLED_ERR_BATCH_TOO_LARGE;
  }
  const int rows = cu_rows[n_reqs];
  if (cu_rows[0] != 0 || rows < n_reqs) return SLED_ERR_ARG;
  if (rows > kMaxRows) {
    std::fprintf(stderr, "sled_accept_rows_static: %d rows exceed the fixed maximum of %d\n", rows, kMaxRows);
    return SLED_ERR_BATCH_TOO_LARGE;
  }
  if (rows > n_reqs && (!drafts || (!greedy && !q_rows))) return SLED_ERR_ARG;   // draft ids are read in both modes
  for (int i = 0; i < n_reqs; ++i)
    if (cu_rows[i + 1] - cu_rows[i] < 1) return SLED_ERR_ARG;                      // checked before anything is written
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev == 0) { cudaGetLastError(); return SLED_ERR_NO_DEVICE; }
  {
    // the kernel runs on the current device: the logits must live there (the array's address is per device)
    int cur = -1;
    cudaPointerAttributes attr{};
    if (cudaGetDevice(&cur) != cudaSuccess) return SLED_ERR_NO_DEVICE;
    const bool ok = cudaPointerGetAttributes(&attr, logits) == cudaSuccess && attr.type == cudaMemoryTypeDevice &&
                    attr.device == cur;
    cudaGetLastError();
    if (!ok) return SLED_ERR_ARG;
  }
  StaticBlock* dev = nullptr;
  int rc = block_address(&dev);
  if (rc) return rc;

  // host image of the block, built on the stack (nothing is allocated on either side): that much of the caller's stack
  StaticBlock host;
  std::memset(&host, 0, sizeof(host));  // rows the kernel never reads and old results start from zero
  int64_t drow = 0;
  for (int i = 0; i < n_reqs; ++i) {
    const int k = cu_rows[i + 1] - cu_rows[i] - 1;
    for (int j = 0; j < k; ++j) {
      const int d = drafts[drow + j];
      if (d < 0 || d >= vocab) return SLED_ERR_TOKEN_RANGE;
      host.ids[cu_rows[i] + 1 + j] = d;
    }
    host.qptr[i] = (q_rows && k > 0) ? q_rows + drow * vocab : nullptr;
    drow += k;
    host.cu[i] = cu_rows[i];
    host.lo[i] = static_cast<uint32_t>(ctx_ids[i]);
    host.hi[i] = static_cast<uint32_t>(ctx_ids[i] >> 32);
    host.pos0[i] = static_cast<int32_t>(pos0[i]);
  }
  host.cu[n_reqs] = rows;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the array keeps the previous call's contents: the whole block is overwritten, results included
  cudaError_t err = cudaMemcpyAsync(dev, &host, sizeof(host), cudaMemcpyHostToDevice, s);
  sled::AcceptArgs aa{};
  aa.logits = logits;
  aa.cu_q = dev->cu;           // addresses inside the device block (computed, not read, on the host)
  aa.ids = dev->ids;
  aa.q_rows = greedy ? nullptr : dev->qptr;
  aa.ctx_lo = dev->lo;
  aa.ctx_hi = dev->hi;
  aa.pos0 = dev->pos0;
  aa.results = dev->results;
  aa.B = n_reqs;
  aa.V = vocab;
  aa.inv_tau = 1.0f / temperature;
  aa.greedy = greedy ? 1 : 0;
  aa.seed = seed;
  int n = err == cudaSuccess ? sled::launch_accept(aa, s) : -1;
  if (err == cudaSuccess)
    err = cudaMemcpyAsync(host.results, dev->results, sizeof(int32_t) * 3 * n_reqs, cudaMemcpyDeviceToHost, s);
  if (err == cudaSuccess) err = cudaStreamSynchronize(s);
  if (err == cudaSuccess) err = cudaGetLastError();
  if (err != cudaSuccess || n < 0) {
    std::fprintf(stderr, "sled_accept_rows_static failed: %s\n", cudaGetErrorString(err));
    return n < 0 && err == cudaSuccess ? SLED_ERR_ARG : SLED_ERR_DEVICE;
  }
  for (int i = 0; i < n_reqs; ++i) {
    results[i].n_accepted = host.results[3 * i];
    results[i].next_token = host.results[3 * i + 1];
    results[i].status = host.results[3 * i + 2];
  }
  return SLED_OK;
}
