// Shared host/device helpers for the decode-step kernels.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <math.h>
#include <mutex>

#include "../../include/grace.h"

#define GRACE_CUDA_TRY(expr)                                  \
  do {                                                        \
    cudaError_t _e = (expr);                                  \
    if (_e != cudaSuccess) return GRACE_CUDA_ERROR;           \
  } while (0)

// Follows every kernel launch: counts it (grace_kernel_launch_count) and checks the launch.
extern unsigned long long g_grace_launches;
#define GRACE_LAUNCH_CHECK()                                  \
  do {                                                        \
    __atomic_fetch_add(&g_grace_launches, 1ull, __ATOMIC_RELAXED); \
    if (cudaGetLastError() != cudaSuccess) return GRACE_CUDA_ERROR; \
  } while (0)

static inline bool grace_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

namespace grace {

constexpr uint32_t kFullMask = 0xffffffffu;
constexpr uint32_t kKeyNegInf = 0x007fffffu;   // ordered key of -inf

// Monotone map fp32 -> uint32: larger value <=> larger key.  -0.0 maps with +0.0.
__device__ __forceinline__ uint32_t ordered_key(float x) {
  uint32_t b = __float_as_uint(x);
  if (b == 0x80000000u) b = 0u;
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// One 32-byte store (a whole sector; the address must be 32-byte aligned).
__device__ __forceinline__ void st_global_32B(void* p, const uint4& lo, const uint4& hi) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"l"(p), "r"(lo.x), "r"(lo.y), "r"(lo.z), "r"(lo.w), "r"(hi.x), "r"(hi.y), "r"(hi.z), "r"(hi.w) : "memory");
}

__device__ __forceinline__ void flag_status(int32_t* d_status, int bits) {
  if (d_status != nullptr) atomicOr(d_status, bits);
}

// splitmix64 finaliser used by the prefix Bloom filter.
__host__ __device__ __forceinline__ uint64_t mix64(uint64_t key) {
  uint64_t z = key + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__device__ __forceinline__ float bf16_lo(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t packed) { return __uint_as_float(packed & 0xffff0000u); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// 16-byte read-only load that does not allocate in L1 (data read once per kernel)
__device__ __forceinline__ uint4 ld_stream_u4(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// Packed pairs of fp32 (sm_100 executes add/mul/fma on two fp32 lanes per instruction).
typedef unsigned long long f32x2_t;
__device__ __forceinline__ f32x2_t f2_pack(float lo, float hi) {
  f32x2_t r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi)); return r;
}
__device__ __forceinline__ void f2_unpack(f32x2_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// the two bf16 halves of a 32-bit word, widened: (low half, high half)
__device__ __forceinline__ f32x2_t f2_from_bf16x2(uint32_t w) {
  f32x2_t r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(w << 16), "r"(w & 0xffff0000u)); return r;
}
__device__ __forceinline__ f32x2_t f2_add(f32x2_t a, f32x2_t b) {
  f32x2_t r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r;
}
__device__ __forceinline__ f32x2_t f2_sub(f32x2_t a, f32x2_t b) {
  f32x2_t r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r;
}
__device__ __forceinline__ f32x2_t f2_mul(f32x2_t a, f32x2_t b) {
  f32x2_t r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r;
}
__device__ __forceinline__ f32x2_t f2_fma(f32x2_t a, f32x2_t b, f32x2_t c) {
  f32x2_t r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c)); return r;
}

// Programmatic dependent launch: a kernel launched with launch_pdl may be scheduled while the kernel
// before it in the stream is still draining; it must call pdl_wait() before its first access to global
// memory that an earlier kernel wrote or still reads (the wait returns once every earlier kernel has
// completed and its writes are visible).  pdl_trigger() lets the NEXT kernel start being scheduled.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// One-time per-device set-up (kernel attributes, occupancy figures and symbol addresses are per device).
//     static unsigned long long done_devices = 0;
//     DeviceSetup su(&done_devices);
//     if (su) { ...set-up for the calling thread's current device...; su.done(); }
// The first caller on a device runs the set-up under a process-wide mutex and publishes the device's
// bit only after it has completed; a second host thread arriving meanwhile waits for the mutex and then
// finds the bit set.  A set-up that returns early (an error) leaves the bit clear and is retried.
constexpr int kMaxDevices = 64;
inline std::mutex& device_setup_mutex() { static std::mutex m; return m; }
struct DeviceSetup {
  unsigned long long* mask;
  unsigned long long bit;
  int dev;
  bool needed;
  std::unique_lock<std::mutex> lock;
  explicit DeviceSetup(unsigned long long* m) : mask(m), bit(0), dev(0), needed(true) {
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { dev = 0; return; }   // set up, never cached
    bit = 1ull << dev;
    if (__atomic_load_n(mask, __ATOMIC_ACQUIRE) & bit) { needed = false; return; }
    lock = std::unique_lock<std::mutex>(device_setup_mutex());
    needed = !(__atomic_load_n(mask, __ATOMIC_ACQUIRE) & bit);
  }
  explicit operator bool() const { return needed; }
  void done() { if (bit) __atomic_fetch_or(mask, bit, __ATOMIC_RELEASE); }
};
inline int current_device_index() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
  return dev;
}

}  // namespace grace
