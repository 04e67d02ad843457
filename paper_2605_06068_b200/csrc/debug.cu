// Diagnostic kernels behind the pda_debug_* entry points: the bounded waits made to run out on purpose
// (a barrier nobody arrives at -- nothing faults, nothing waits without a limit), and a read-only
// streaming probe that gives the practical ceiling for a kernel that only reads HBM.
#include "common.cuh"
#include "tma_ptx.cuh"
#include "tcgen05_ptx.cuh"

namespace pda {

namespace {

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// One warp initialises an mbarrier that expects one arrival, never arrives, and runs the two bounded
// waits of the attention kernels on it with `polls` as their limit. Both must come back false; the
// kernel then records PDA_DEV_TIMEOUT exactly as the attention kernels do and returns.
// result[0], result[1]: nanoseconds the suspended (try_wait) and the spinning (test_wait) wait took;
// result[2]: bit 0 / bit 1 set if the respective wait claimed the phase had completed (it must not).
__global__ void __launch_bounds__(32) wait_timeout_kernel(uint32_t polls, int32_t* status, uint64_t* result) {
  __shared__ __align__(8) uint64_t bar_storage;
  const uint32_t bar = smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    fence_mbar_init();
  }
  __syncwarp();
  const uint64_t t0 = global_ns();
  const bool ok_a = __all_sync(0xffffffffu, mbar_wait_bounded(bar, 0, polls));
  const uint64_t t1 = global_ns();
  const bool ok_b = __all_sync(0xffffffffu, mbar_spin_bounded(bar, 0, polls));
  const uint64_t t2 = global_ns();
  if (threadIdx.x == 0) {
    if (!ok_a || !ok_b) report(status, PDA_DEV_TIMEOUT);
    if (result != nullptr) {
      result[0] = t1 - t0;
      result[1] = t2 - t1;
      result[2] = (ok_a ? 1u : 0u) | (ok_b ? 2u : 0u);
    }
  }
}

constexpr int kProbeThreads = 256;
constexpr int kProbeUnroll = 8;  // independent 16-byte loads in flight per thread

// Every CTA strides through the buffer with 16-byte loads that bypass L1 and folds what it reads into
// one word, so that the loads cannot be dropped; nothing is written but one word per CTA.
__global__ void __launch_bounds__(kProbeThreads) read_probe_kernel(const uint4* __restrict__ buf, size_t n_vec,
                                                                   uint32_t* __restrict__ sink) {
  const size_t stride = static_cast<size_t>(gridDim.x) * kProbeThreads;
  size_t i = static_cast<size_t>(blockIdx.x) * kProbeThreads + threadIdx.x;
  uint32_t acc = 0;
  for (; i + (kProbeUnroll - 1) * stride < n_vec; i += kProbeUnroll * stride) {
    uint4 v[kProbeUnroll];
#pragma unroll
    for (int k = 0; k < kProbeUnroll; ++k) {
      const uint4* ptr = buf + i + k * stride;
      asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                   : "=r"(v[k].x), "=r"(v[k].y), "=r"(v[k].z), "=r"(v[k].w) : "l"(ptr));
    }
#pragma unroll
    for (int k = 0; k < kProbeUnroll; ++k) acc ^= v[k].x ^ v[k].y ^ v[k].z ^ v[k].w;
  }
  for (; i < n_vec; i += stride) {
    const uint4 v = __ldg(buf + i);
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0 && acc == 0x9e3779b9u) atomicAdd(sink, 1u);  // (practically never: keeps the loads live)
}

}  // namespace

cudaError_t launch_wait_timeout(uint32_t polls, int32_t* status, uint64_t* result, cudaStream_t stream) {
  wait_timeout_kernel<<<1, 32, 0, stream>>>(polls, status, result);
  return cudaGetLastError();
}

cudaError_t launch_read_probe(const void* buf, size_t bytes, uint32_t* sink, cudaStream_t stream) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  // 8 CTAs of 256 threads per SM: 2048 threads x 8 loads x 16 B = 256 KB in flight per SM
  read_probe_kernel<<<sms * 8, kProbeThreads, 0, stream>>>(static_cast<const uint4*>(buf), bytes / 16, sink);
  return cudaGetLastError();
}

}  // namespace pda
