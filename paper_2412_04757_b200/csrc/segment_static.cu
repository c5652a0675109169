// Allocation-free variant of the span segmenter.
//
// Some callers cannot obtain device memory at the point where they need a segmentation: code running inside a
// memory-pool-managed region where every byte is already spoken for, plugins loaded into a host process that
// forbids cudaMalloc after start-up, or a latency-critical service thread that must not touch the allocator.
// ltri_segment_map_static gives them the segmenter with its scratch (the row-suffix-sum table and the
// anti-diagonal candidates) in a fixed device array that is part of the library image, so the call needs no
// context, no arena and no allocation of any kind.  The price is a modest size limit and a shared scratch.
#include <mutex>

#include "../../include/ltri.h"
#include "common.cuh"

namespace {

using namespace ltri;

constexpr int kStaticMaxM = LTRI_STATIC_SEGMENT_MAX_M;  // largest map side the static scratch can hold
constexpr int kStaticJmax = 2 * kMaxTopK + 1;

// byte offsets inside the scratch array (each 256-byte aligned)
constexpr size_t kOffRsuf = 0;
constexpr size_t kOffBest = kOffRsuf + sizeof(long long) * kStaticMaxM * kStaticMaxM;
constexpr size_t kOffTheta = kOffBest + sizeof(long long) * 2 * kStaticMaxM;
constexpr size_t kOffPendStart = kOffTheta + 256;
constexpr size_t kOffPendLen = kOffPendStart + 1024;
constexpr size_t kOffPendCnt = kOffPendLen + 1024;
constexpr size_t kOffJcnt = kOffPendCnt + 256;
constexpr size_t kOffStatus = kOffJcnt + 256;
constexpr size_t kScratchBytes = kOffStatus + 256;
static_assert(kStaticJmax * sizeof(int) <= 1024, "pending-span area too small");

// Every GPU that loads the library holds this array (about 0.5 MiB) until the process exits.  In host code the
// name below is only a handle: the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_seg_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// interleave the segmenter's {start[], len[]} arrays into the caller's {start,len} pairs
// (status: the word the segmenter's device-side checks write; a failed check is reported through *n_out)
__global__ void k_pack_spans(const int* __restrict__ start, const int* __restrict__ len, const int* __restrict__ cnt,
                             const int* __restrict__ status, int cap_pairs, int32_t* __restrict__ pairs,
                             int32_t* __restrict__ n_out) {
  const int code = *status;
  if (code != 0) {
    if (threadIdx.x == 0) *n_out = (code <= LTRI_EINVAL && code >= LTRI_ETIMEOUT) ? code : LTRI_EDEVICE;
    return;
  }
  const int n = *cnt;
  for (int i = threadIdx.x; i < n && i < cap_pairs; i += blockDim.x) {
    pairs[2 * i] = start[i];
    pairs[2 * i + 1] = len[i];
  }
  if (threadIdx.x == 0) *n_out = n;
}

}  // namespace

extern "C" int ltri_segment_map_static(const int32_t* Mq, int m, int64_t theta_q, int max_spans, int32_t* pairs,
                                       int cap_pairs, int32_t* n_out, void* cuda_stream) {
  if (!Mq || !pairs || !n_out || m < 1 || max_spans < 1 || cap_pairs < 1) return LTRI_EINVAL;
  if (m > kStaticMaxM || max_spans > kMaxTopK) return LTRI_ECAPACITY;  // beyond the fixed scratch
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return LTRI_ECUDA;
  if (dev < 0 || dev >= kMaxDevices) return LTRI_ECAPACITY;
  {
    // the scratch used below is the current device's: a map that the runtime knows to live on another device would
    // be read across devices (or not at all), so it is refused here; pointers the runtime cannot attribute pass
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, Mq) == cudaSuccess) {
      if (attr.type == cudaMemoryTypeDevice && attr.device != dev) return LTRI_EINVAL;
    } else {
      cudaGetLastError();
    }
  }
  unsigned char* base = nullptr;
  {
    // first call on this device: resolve the device address of the scratch array (not capturable work)
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_seg_scratch) != cudaSuccess || !p) return LTRI_ECUDA;
      g_scratch_addr[dev] = p;
    }
    base = static_cast<unsigned char*>(g_scratch_addr[dev]);
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // a one-layer, one-sequence view whose buffers are the caller's map and the static scratch
  DevCtx c = {};
  c.NL = 1;
  c.NS = 1;
  c.Hq = c.Hkv = c.G = 1;
  c.chunk = m;  // leading dimension of the caller's dense [m][m] map
  c.C = max_spans;
  c.Jmax = kStaticJmax;
  c.slots = 1;
  c.reps = 1;
  c.Mq = const_cast<int*>(reinterpret_cast<const int*>(Mq));
  c.Rsuf = reinterpret_cast<long long*>(base + kOffRsuf);
  c.best = reinterpret_cast<long long*>(base + kOffBest);
  c.thetaq = reinterpret_cast<long long*>(base + kOffTheta);
  c.pend_start = reinterpret_cast<int*>(base + kOffPendStart);
  c.pend_len = reinterpret_cast<int*>(base + kOffPendLen);
  c.pend_cnt = reinterpret_cast<int*>(base + kOffPendCnt);
  c.Jcnt = reinterpret_cast<int*>(base + kOffJcnt);
  c.status = reinterpret_cast<int*>(base + kOffStatus);
  // the scratch keeps the previous call's contents: the status words and the span count must start at zero
  // (the candidate table is cleared by the segmenter itself)
  if (cudaMemsetAsync(base + kOffPendCnt, 0, kScratchBytes - kOffPendCnt, st) != cudaSuccess) return LTRI_ECUDA;
  if (launch_segment(c, 0, 0, 1, m, 0, 0, /*theta_mode=*/0, 0.f, theta_q, max_spans, 0, 0, nullptr, st) != cudaSuccess)
    return LTRI_ECUDA;
  k_pack_spans<<<1, 128, 0, st>>>(c.pend_start, c.pend_len, c.pend_cnt, c.status, cap_pairs, pairs, n_out);
  return cudaGetLastError() == cudaSuccess ? LTRI_OK : LTRI_ECUDA;
}
