// Burst/gap store microbenchmark on this GPU's own HBM: the paper's periodic-burst and isolated-burst
// patterns (Sec. 3.1) run against local memory, i.e. its "local-memory control".  K producers (one CTA of
// 128 threads per SM, the width of the GEMM epilogue) each issue B bytes of 16-byte stores, then spin for
// G clocks without storing; the sender-visible issue span of every burst is taken with clock64().
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/xstage.h"

namespace {

constexpr int kProbeThreads = 128;
constexpr long long kStartBudget = 2000000000LL;   // clocks a producer waits for the others at the aligned start
constexpr long long kMaxGapBudget = 4000000000LL;  // gap_clocks x periods may not exceed this (about 2 s of spinning)

struct ProbeHeader {
  int arrived;        // producers that reached the start line
  int timed_out;      // set when a producer gave up waiting
  long long clk0, clk1;         // clock64 of producer 0 at start / end
  unsigned long long ns0, ns1;  // globaltimer of producer 0 at start / end
};

__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__global__ void __launch_bounds__(kProbeThreads, 1)
store_burst_probe(uint4* __restrict__ buffer, long long vec_per_producer, long long vec_per_burst, long long gap_clocks,
                  int periods, ProbeHeader* hdr, long long* issue_clk, long long* period_clk) {
  extern __shared__ unsigned char occupancy_pad[];   // only there to keep one producer per SM
  __shared__ int go;
  const int tid = threadIdx.x, producer = blockIdx.x, K = gridDim.x;
  if (tid == 0) {
    go = 1;
    atomicAdd(&hdr->arrived, 1);
    const long long t0 = clock64();
    while (atomicAdd(&hdr->arrived, 0) < K) {     // aligned start; bounded
      if (clock64() - t0 > kStartBudget || atomicAdd(&hdr->timed_out, 0)) {
        atomicExch(&hdr->timed_out, 1);
        go = 0;
        break;
      }
    }
    if (producer == 0) {
      hdr->clk0 = clock64();
      hdr->ns0 = globaltimer_ns();
    }
  }
  __syncthreads();
  if (!go) return;
  uint4* mine = buffer + static_cast<long long>(producer) * vec_per_producer;
  long long cursor = 0;
  long long t_period_start = clock64();
  for (int n = 0; n < periods; ++n) {
    if (cursor + vec_per_burst > vec_per_producer) cursor = 0;
    const uint4 val = make_uint4(n, producer, tid, 0x5A5A5A5Au);
    __syncthreads();
    const long long t0 = clock64();
#pragma unroll 1   // the same loop body for every burst size
    for (long long v = tid; v < vec_per_burst; v += kProbeThreads) mine[cursor + v] = val;
    __syncthreads();                                   // every thread of the producer has issued its stores
    const long long t1 = clock64();
    cursor += vec_per_burst;
    while (clock64() - t1 < gap_clocks) { }            // the gap: no stores
    const long long t2 = clock64();
    if (tid == 0) {
      issue_clk[static_cast<long long>(n) * K + producer] = t1 - t0;
      period_clk[static_cast<long long>(n) * K + producer] = t2 - t_period_start;
    }
    t_period_start = t2;
  }
  if (tid == 0 && producer == 0) {
    hdr->clk1 = clock64();
    hdr->ns1 = globaltimer_ns();
  }
}

}  // namespace

extern "C" int xstage_store_probe(int32_t producers, int64_t bytes_per_burst, int64_t gap_clocks, int32_t periods,
                                  void* device_buffer, uint64_t buffer_bytes, double* issue_mean_clocks,
                                  double* issue_max_clocks, double* period_mean_clocks, double* clocks_per_us,
                                  void* stream) {
  if (producers < 1 || bytes_per_burst < 16 || bytes_per_burst % 16 != 0 || gap_clocks < 0 || periods < 1 ||
      periods > 65536 || !device_buffer || !issue_mean_clocks || !period_mean_clocks)
    return -1;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return -2;
  if (producers > sms) return -1;                      // one resident producer per SM, or the start line never fills
  // the gaps are busy-waits on every SM: a gap given in the wrong unit must not occupy a shared GPU for minutes
  if (gap_clocks > kMaxGapBudget / periods) return -1;
  const long long vec_per_burst = bytes_per_burst / 16;
  const long long vec_per_producer = static_cast<long long>(buffer_bytes / 16) / producers;
  if (vec_per_producer < vec_per_burst || (reinterpret_cast<uintptr_t>(device_buffer) & 15u)) return -1;

  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const size_t n = static_cast<size_t>(periods) * producers;
  unsigned char* d_res = nullptr;
  if (cudaMalloc(&d_res, sizeof(ProbeHeader) + 2 * n * sizeof(long long)) != cudaSuccess) return -2;
  ProbeHeader* d_hdr = reinterpret_cast<ProbeHeader*>(d_res);
  long long* d_issue = reinterpret_cast<long long*>(d_res + sizeof(ProbeHeader));
  long long* d_period = d_issue + n;
  int rc = 0;
  const int pad = 120 * 1024;                          // more than half an SM's shared memory: one CTA per SM
  std::vector<long long> h_issue(n), h_period(n);
  ProbeHeader h{};
  if (cudaMemsetAsync(d_res, 0, sizeof(ProbeHeader) + 2 * n * sizeof(long long), cs) != cudaSuccess ||
      cudaFuncSetAttribute(store_burst_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, pad) != cudaSuccess) {
    rc = -2;
  } else {
    store_burst_probe<<<producers, kProbeThreads, pad, cs>>>(static_cast<uint4*>(device_buffer), vec_per_producer,
                                                            vec_per_burst, gap_clocks, periods, d_hdr, d_issue,
                                                            d_period);
    if (cudaMemcpyAsync(&h, d_hdr, sizeof(h), cudaMemcpyDeviceToHost, cs) != cudaSuccess ||
        cudaMemcpyAsync(h_issue.data(), d_issue, n * sizeof(long long), cudaMemcpyDeviceToHost, cs) != cudaSuccess ||
        cudaMemcpyAsync(h_period.data(), d_period, n * sizeof(long long), cudaMemcpyDeviceToHost, cs) != cudaSuccess ||
        cudaStreamSynchronize(cs) != cudaSuccess)
      rc = -2;
    else if (h.timed_out)
      rc = -3;
  }
  cudaFree(d_res);
  if (rc != 0) return rc;
  for (int p = 0; p < periods; ++p) {
    double si = 0, sp = 0, mx = 0;
    for (int k = 0; k < producers; ++k) {
      const double vi = static_cast<double>(h_issue[static_cast<size_t>(p) * producers + k]);
      si += vi;
      sp += static_cast<double>(h_period[static_cast<size_t>(p) * producers + k]);
      if (vi > mx) mx = vi;
    }
    issue_mean_clocks[p] = si / producers;
    period_mean_clocks[p] = sp / producers;
    if (issue_max_clocks) issue_max_clocks[p] = mx;
  }
  if (clocks_per_us) {
    const double ns = static_cast<double>(h.ns1 - h.ns0);
    *clocks_per_us = ns > 0 ? static_cast<double>(h.clk1 - h.clk0) / ns * 1e3 : 0.0;
  }
  return 0;
}
