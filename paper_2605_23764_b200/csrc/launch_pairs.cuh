// Launch of a persistent kernel on clusters of two CTAs (one CTA per SM).  The opt-in shared-memory
// size is a per-device function attribute and the number of CTA pairs that can be resident together
// depends on the device, so both are kept per device, under a lock: contexts on different GPUs of
// one process, and host threads, may launch at the same time.
#pragma once

#include <cuda_runtime.h>
#include <string.h>

#include <mutex>

namespace moe {

constexpr int MAX_DEVICES = 64;

struct PairLaunchState {
  std::mutex mu;
  bool attr_set[MAX_DEVICES] = {};
  int max_pairs[MAX_DEVICES] = {};
};

template <class Kernel, class Args>
cudaError_t launch_on_pairs(PairLaunchState& st, Kernel kernel, const Args& args, int threads, size_t smem_bytes,
                            int num_sms, bool cooperative, cudaStream_t s) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3((num_sms / 2) * 2);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeCooperative;  // the launch fails rather than run with CTAs that are not all resident
  attr[1].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = cooperative ? 2 : 1;
  int pairs = 0;
  {
    std::lock_guard<std::mutex> lock(st.mu);
    if (!st.attr_set[dev]) {
      e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
      if (e != cudaSuccess) return e;
      st.attr_set[dev] = true;
    }
    if (st.max_pairs[dev] == 0) {   // CTA pairs that can be resident together (SMs pair up inside a GPC)
      int n = 0;
      e = cudaOccupancyMaxActiveClusters(&n, kernel, &cfg);
      if (e != cudaSuccess) return e;
      st.max_pairs[dev] = n > 0 ? n : 1;
    }
    pairs = st.max_pairs[dev];
  }
  if (2 * pairs < (int)cfg.gridDim.x) cfg.gridDim = dim3(2 * pairs);
  return cudaLaunchKernelEx(&cfg, kernel, args);
}

}  // namespace moe
