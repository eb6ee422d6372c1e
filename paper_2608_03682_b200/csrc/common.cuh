// Shared declarations of the CUDA path: device-side request block, status word, activation
// layouts and small math helpers.  Nothing here is used by (or shared with) the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace phyai {

// ---------------------------------------------------------------------------------------------
// Status word (device memory, one per handle).  Kernels return immediately when it is non-zero,
// so a failed validation or an expired wait turns the rest of the enqueued loop into no-ops.
// ---------------------------------------------------------------------------------------------
enum : int { ST_OK = 0, ST_INVALID_ARG = 1, ST_TIMEOUT = 5 };

__device__ __forceinline__ bool status_set(const int* status) {
  return *reinterpret_cast<const volatile int*>(status) != 0;
}

// ---------------------------------------------------------------------------------------------
// Programmatic dependent launch.  Kernels of the per-operator loop are launched with the "programmatic stream
// serialization" attribute: the next kernel's CTAs may be scheduled (and run their set-up) while this kernel
// drains.  Every such kernel calls pdl_enter() before its first global-memory access: it lets its own dependents
// start early and then waits until the kernels it depends on have completed and their writes are visible.  In a
// launch without the attribute both instructions are no-ops.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------
// Tracing aid (the paper times phases with GPU-side profiler scopes): with tracing switched on, one CTA of each
// traced launch writes device-global-timer stamps (ns) into its 16-entry slot of a trace buffer.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void trace_stamp(unsigned long long* slot, int i) {
  if (slot) slot[i] = global_ns();
}

// ---------------------------------------------------------------------------------------------
// Request block: written by a tiny kernel right before each denoise call, read by every kernel
// of the loop.  Keeping the per-request pointers and lengths here (not in kernel arguments) lets
// one captured CUDA graph serve every request of the same (batch, n_steps).
// ---------------------------------------------------------------------------------------------
struct Request {
  const void* prefix_kv;   // [L][2][kv_tokens][Hkv][dh], fp32 or bf16
  uint64_t kv_tokens;      // token capacity of prefix_kv (stride between K and V planes)
  const int* cu_lens;      // device [batch+1]
  const float* states;     // [batch][Ds] or null
  const float* noise;      // [batch][H][A]
  float* x;                // [batch][H][A]: the Euler state, = out_actions
  int batch;
  int single_len;          // prefix_len of the single-request entry point
};

// ---------------------------------------------------------------------------------------------
// Activation layouts.
//   Row-major fp32 [rows][cols] for the residual stream and the CUDA-core path.
//   "Tiled bf16" for every tensor-core GEMM input: [cols/64][rows_pad][64] with the eight 16-byte
//   chunks of each 128-byte row XOR-swizzled by (row & 7).  A tile of NT rows x 64 columns is then
//   one contiguous NT*128-byte block that is already the 128-byte-swizzled K-major shared-memory
//   image tcgen05.mma expects, so it is fetched with one bulk copy and no tensor map.
// ---------------------------------------------------------------------------------------------
__host__ __device__ __forceinline__ size_t tiled_index(int row, int col, int rows_pad) {
  const int kc = col >> 6, within = col & 63;
  const int chunk = (within >> 3) ^ (row & 7);
  return ((size_t)kc * rows_pad + row) * 64 + (size_t)chunk * 8 + (within & 7);
}

// Row order of the packed fused-QKV weight matrix.  Inside every q / k head the dh channels are
// arranged so that each 128-row tile holds 64 channels of the first half of the head followed by
// their 64 rotary partners (channel + dh/2): a GEMM epilogue then finds both members of a rotary pair
// in one accumulator tile, 64 rows apart.  The v region and heads of <= 128 channels keep their order.
__host__ __device__ __forceinline__ int qkv_channel_to_packed(int c, int dh) {
  if (dh <= 128) return c;
  const int hb = c - c % dh, w = c % dh, half = dh >> 1;
  const int t = (w % half) >> 6, r = (w & 63) + (w >= half ? 64 : 0);
  return hb + t * 128 + r;
}
__host__ __device__ __forceinline__ int qkv_packed_to_channel(int n, int dh) {
  if (dh <= 128) return n;
  const int hb = n - n % dh, w = n % dh, half = dh >> 1;
  const int t = w >> 7, r = w & 127;
  return hb + (r < 64 ? t * 64 + r : half + t * 64 + (r - 64));
}

struct RowMajorF32 {
  float* p;
  int ld;
  __device__ __forceinline__ void store(int row, int col, float v) const { p[(size_t)row * ld + col] = v; }
};
struct TiledBf16 {
  __nv_bfloat16* p;
  int rows_pad;
  __device__ __forceinline__ void store(int row, int col, float v) const {
    p[tiled_index(row, col, rows_pad)] = __float2bfloat16_rn(v);
  }
};

// ---------------------------------------------------------------------------------------------
// math helpers (fp32)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float swish_f(float z) { return z / (1.0f + __expf(-z)); }
__device__ __forceinline__ float swish_precise(float z) { return z / (1.0f + expf(-z)); }

__device__ __forceinline__ float gelu_tanh_f(float z) {
  const float k = 0.7978845608028654f;  // sqrt(2/pi)
  const float u = k * (z + 0.044715f * z * z * z);
  return 0.5f * z * (1.0f + tanhf(u));
}
__device__ __forceinline__ float gelu_erf_f(float z) { return 0.5f * z * (1.0f + erff(z * 0.7071067811865476f)); }
__device__ __forceinline__ float gelu_f(float z, int exact) { return exact ? gelu_erf_f(z) : gelu_tanh_f(z); }

// GELU for the GeGLU epilogues: tanh form written as z * sigmoid(2u) (one exp, one fast divide), erf form as is.
__device__ __forceinline__ float gelu_fast(float z, int exact) {
  if (exact) return gelu_erf_f(z);
  // 0.5 z (1 + tanh(u)), u = sqrt(2/pi) (z + 0.044715 z^3), with the hardware tanh (absolute error ~5e-4 of a
  // factor in [0, 2]: far inside the bf16 rounding of the result)
  const float u = z * fmaf(0.7978845608028654f * 0.044715f, z * z, 0.7978845608028654f);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
  const float hz = 0.5f * z;
  return fmaf(hz, t, hz);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

}  // namespace phyai
