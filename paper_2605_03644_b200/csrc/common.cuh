// Shared host/device helpers of the adapshot CUDA library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "adapshot.h"

#define ADAPSHOT_VERSION_NUMBER 100

#define ADS_CHECK_CUDA(expr)                              \
  do {                                                    \
    cudaError_t e__ = (expr);                             \
    if (e__ != cudaSuccess) return ADAPSHOT_ECUDA;        \
  } while (0)

static inline bool ads_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t ads_round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// A launch failure is reported as ADAPSHOT_ECUDA without clearing anything else.
static inline int ads_launch_status() {
  return cudaGetLastError() == cudaSuccess ? ADAPSHOT_OK : ADAPSHOT_ECUDA;
}

// Per-device host-side caches: a process may drive several GPUs, and both the SM count and a
// kernel's shared-memory attribute belong to the device that is current at the call.
constexpr int kAdsMaxDevices = 64;
static inline int ads_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kAdsMaxDevices) return -1;
  return dev;
}
// SM count of the current device (0 on error); looked up once per device.
static inline int ads_sm_count() {
  static int n_sm[kAdsMaxDevices] = {0};
  const int dev = ads_current_device();
  if (dev < 0) return 0;
  if (n_sm[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 0;
    n_sm[dev] = n;
  }
  return n_sm[dev];
}
// Raises a kernel's dynamic shared-memory limit once per device.  `done` is a per-kernel table
// (kAdsMaxDevices entries) owned by the caller.  The value is the same every time, so two
// threads that race here both write it.
template <typename Kernel>
static inline int ads_set_max_smem(Kernel kernel, int bytes, bool* done) {
  const int dev = ads_current_device();
  if (dev < 0) return ADAPSHOT_ECUDA;
  if (!done[dev]) {
    ADS_CHECK_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    done[dev] = true;
  }
  return ADAPSHOT_OK;
}

// Device: record an error code once; later codes do not overwrite the first.
__device__ __forceinline__ void ads_set_status(int32_t* status, int32_t code) {
  if (status != nullptr) atomicCAS(status, 0, code);
}

// Order-preserving map of an fp64 score to an unsigned key; larger score -> SMALLER key so that an
// ascending order on (key, id) lists the most relevant shot first and equal scores by ascending id.
__device__ __forceinline__ unsigned long long ads_desc_key(double s) {
  unsigned long long u = (unsigned long long)__double_as_longlong(s);
  u = (u >> 63) ? ~u : (u | 0x8000000000000000ull);   // ascending in s
  return ~u;
}
__device__ __forceinline__ double ads_key_score(unsigned long long k) {
  unsigned long long u = ~k;
  u = (u >> 63) ? (u & 0x7fffffffffffffffull) : ~u;
  return __longlong_as_double((long long)u);
}

// Top k of N candidates per query from their sort keys (select.cu): keys [B][N] as ads_desc_key
// writes them, ids [B][N] = 0..N-1 (read only when N needs the chunked sort), cand = scratch of
// ads_topk_scratch_bytes(N, B, k) bytes.  Enqueues on st; returns an ADAPSHOT_* code.
size_t ads_topk_scratch_bytes(int N, int B, int k);
int ads_topk_from_keys(const unsigned long long* keys, const int* ids, int N, int B, int k, void* cand,
                       int32_t* sel_idx, float* sel_score, cudaStream_t st);

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// Angle p * theta_i formed in fp64 and reduced to [-pi, pi] before the fp32
// sincos, so that the result keeps fp32 accuracy at positions of 64K and more.
__device__ __forceinline__ float rope_reduced_angle(double delta, double theta) {
  const double kInv2Pi = 0.15915494309189533577;
  const double k2PiHi = 6.283185307179586232;
  const double k2PiLo = 2.449293598294706354e-16;
  double a = delta * theta;
  double n = rint(a * kInv2Pi);
  double r = fma(-n, k2PiHi, a);
  r = fma(-n, k2PiLo, r);
  return static_cast<float>(r);
}
__device__ __forceinline__ void rope_sincos(double delta, double theta, float* s, float* c) {
  sincosf(rope_reduced_angle(delta, theta), s, c);
}
// Hardware approximations (absolute error below 1e-6 on [-pi, pi]): for bf16 storage only.
__device__ __forceinline__ void rope_sincos_fast(double delta, double theta, float* s, float* c) {
  const float r = rope_reduced_angle(delta, theta);
  *s = __sinf(r);
  *c = __cosf(r);
}
