// Stand-alone W8A8 projection: the per-token e4m3 quantization kernel and the FP8 tile GEMM of the denoising loop,
// callable on one activation matrix (quantization paragraph: W8A8).  The quantization is a discontinuous step -- a
// whole network with it can only be compared with a reference up to the size of the quantization noise itself --, so
// this entry point is where the arithmetic of the mode is checked exactly: same stored activations in, same codes,
// same scales, and the product to fp32 summation error.
#include <cstdio>

#include "../../include/phyai.h"
#include "kernels.h"

namespace phyai {
namespace {

// tiled e4m3 [K/128][rows_pad][128] -> row-major codes [M][K]
__global__ void k_codes_to_rows(const uint8_t* t, uint8_t* out, int M, int K, int rows_pad) {
  const size_t n = (size_t)M * (K >> 4);
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const int row = (int)(i / (K >> 4)), c16 = (int)(i % (K >> 4));
    const int col = c16 << 4, kc = col >> 7, ch = (col & 127) >> 4;
    const uint4 v = *reinterpret_cast<const uint4*>(t + ((size_t)kc * rows_pad + row) * 128 + ((ch ^ (row & 7)) << 4));
    *reinterpret_cast<uint4*>(out + (size_t)row * K + col) = v;
  }
}

thread_local char op_err[256] = "";
phyai_status_t op_fail(phyai_status_t s, const char* what, cudaError_t e = cudaSuccess) {
  if (e != cudaSuccess) snprintf(op_err, sizeof(op_err), "%s: %s", what, cudaGetErrorString(e));
  else snprintf(op_err, sizeof(op_err), "%s", what);
  return s;
}

}  // namespace
}  // namespace phyai

using namespace phyai;

extern "C" const char* phyai_w8a8_last_error(void) { return op_err; }

extern "C" phyai_status_t phyai_w8a8_project(const void* x_bf16, const uint8_t* w_codes, const float* w_scales, uint32_t M,
                                             uint32_t K, uint32_t N, float* y, uint8_t* x_codes_out, float* x_scales_out,
                                             void* stream) {
  op_err[0] = 0;
  if (!x_bf16 || !w_codes || !w_scales || !y) return op_fail(PHYAI_ERR_INVALID_ARG, "NULL argument");
  if (M == 0 || M > (1u << 16) || K == 0 || K % 128 || K > 4096 || N == 0 || N % 128 || N > (1u << 16))
    return op_fail(PHYAI_ERR_INVALID_ARG, "need 1 <= M <= 65536, K a multiple of 128 up to 4096, N a multiple of 128 up to 65536");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  cudaError_t e = tc_gemm_setup();
  if (e != cudaSuccess) return op_fail(PHYAI_ERR_CUDA, "tc_gemm_setup", e);
  const int rows_pad = (int)((M + 255) / 256 * 256);
  __nv_bfloat16* xt = nullptr;
  uint8_t *xq = nullptr, *wp = nullptr;
  float* xs = nullptr;
  int* status = nullptr;
  auto cleanup = [&]() { cudaFree(xt), cudaFree(xq), cudaFree(wp), cudaFree(xs), cudaFree(status); };
  if ((e = cudaMalloc(&xt, (size_t)rows_pad * K * 2)) != cudaSuccess || (e = cudaMalloc(&xq, (size_t)rows_pad * K)) != cudaSuccess ||
      (e = cudaMalloc(&wp, (size_t)K * N)) != cudaSuccess || (e = cudaMalloc(&xs, (size_t)rows_pad * 4)) != cudaSuccess ||
      (e = cudaMalloc(&status, 4)) != cudaSuccess) {
    cleanup();
    return op_fail(PHYAI_ERR_OOM, "cudaMalloc", e);
  }
  cudaMemsetAsync(xt, 0, (size_t)rows_pad * K * 2, st);
  cudaMemsetAsync(xq, 0, (size_t)rows_pad * K, st);
  cudaMemsetAsync(xs, 0, (size_t)rows_pad * 4, st);
  cudaMemsetAsync(status, 0, 4, st);
  launch_rows_to_tiled(reinterpret_cast<const __nv_bfloat16*>(x_bf16), xt, (int)M, (int)K, rows_pad, st);
  launch_quant_rows(status, xt, xq, xs, rows_pad, (int)M, (int)K, st);
  launch_pack_bytes(w_codes, wp, (int)K, (int)N, 0, st, 0, 0, 0, 1);
  TcGemm g{};
  g.W = reinterpret_cast<const __nv_bfloat16*>(wp), g.X = reinterpret_cast<const __nv_bfloat16*>(xq), g.M = (int)M, g.N = (int)N;
  g.K = (int)K, g.epi = TC_STORE, g.scale = w_scales, g.out_f32 = y, g.ldo = (int)N, g.splits = 1, g.rows_pad = rows_pad;
  g.fp8 = 1, g.xscale = xs, g.wait_limit = 1u << 28;
  e = launch_tc_gemm(status, g, M <= 64 ? 64 : (M <= 1024 ? 128 : 256), st);
  if (e == cudaSuccess && x_codes_out) k_codes_to_rows<<<256, 256, 0, st>>>(xq, x_codes_out, (int)M, (int)K, rows_pad);
  if (e == cudaSuccess && x_scales_out) e = cudaMemcpyAsync(x_scales_out, xs, (size_t)M * 4, cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  int hs = 0;
  if (e == cudaSuccess) e = cudaMemcpy(&hs, status, 4, cudaMemcpyDeviceToHost);
  cleanup();
  if (e != cudaSuccess) return op_fail(PHYAI_ERR_CUDA, "W8A8 projection", e);
  if (hs != 0) return op_fail(PHYAI_ERR_TIMEOUT, "a bounded device-side wait expired");
  return PHYAI_OK;
}
