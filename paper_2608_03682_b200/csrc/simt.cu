// CUDA-core kernels: request block, tables, packing, embedding, norms, the Euler head, a generic
// fp32 GEMM and a generic fp32 attention.  They serve the fp32 configuration end to end (true
// fp32 FMA, no TF32) and provide the small memory-bound steps of the tensor-core path.
#include <cuda_fp8.h>

#include "kernels.h"

namespace phyai {

// =============================================================================================
// request block
// =============================================================================================
__global__ void k_set_request(Request* dst, Request src, int* cu_internal, int* order) {
  if (threadIdx.x == 0) {
    if (src.cu_lens == nullptr) {  // single-request entry point: build cu = {0, prefix_len}
      cu_internal[0] = 0;
      cu_internal[1] = src.single_len;
      src.cu_lens = cu_internal;
      // the walk order of the request-per-CTA kernels: a batched call on the same handle may have left another
      // request index in entry 0
      if (order) order[0] = 0;
    }
    *dst = src;
  }
}
void launch_set_request(Request* dst, const Request& src, int* cu_internal, cudaStream_t st, int* order) {
  k_set_request<<<1, 32, 0, st>>>(dst, src, cu_internal, order);
}

// cu_prefix_lens must be non-decreasing, start >= 0, end <= kv_tokens, differences <= max_prefix.
// Also writes `order`: the requests sorted by descending prefix length (ties by index).  Kernels whose CTAs
// take one request each walk the batch in this order, so the longest requests start first and the grid's tail is short.
__global__ void k_validate(const Request* rq, int* status, int max_prefix, int* order) {
  const int B = rq->batch;
  const int* cu = rq->cu_lens;
  bool bad = false;
  for (int b = threadIdx.x; b < B; b += blockDim.x) {
    const int lo = cu[b], hi = cu[b + 1];
    if (lo < 0 || hi < lo || hi - lo > max_prefix || (uint64_t)hi > rq->kv_tokens) bad = true;
    if (order) {
      const int len = hi - lo;
      int rank = 0;
      for (int c = 0; c < B; ++c) {
        const int lc = cu[c + 1] - cu[c];
        rank += (lc > len || (lc == len && c < b)) ? 1 : 0;
      }
      order[rank] = b;
    }
  }
  if (bad) atomicExch(status, ST_INVALID_ARG);
}
void launch_validate(const Request* rq, int* status, int max_prefix, int* order, cudaStream_t st) {
  k_validate<<<1, 256, 0, st>>>(rq, status, max_prefix, order);
}

// =============================================================================================
// storage decoding
// =============================================================================================
__device__ __forceinline__ float load_src(const void* src, int kind, size_t i) {
  if (kind == 0) return reinterpret_cast<const float*>(src)[i];
  if (kind == 1) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(src)[i]);
  if (kind == 3) {   // int4: two neighbouring elements per byte, the even one in the low nibble; code c = integer c - 8
    const uint8_t b = reinterpret_cast<const uint8_t*>(src)[i >> 1];
    return (float)((int)((i & 1) ? (b >> 4) : (b & 15)) - 8);
  }
  const __half_raw hr = __nv_cvt_fp8_to_halfraw(reinterpret_cast<const __nv_fp8_storage_t*>(src)[i], __NV_E4M3);
  return __half2float(__half(hr));
}

__global__ void k_to_f32(const void* src, int kind, float* dst, size_t n) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = load_src(src, kind, i);
}
void launch_to_f32(const void* src, int kind, float* dst, size_t n, cudaStream_t st) {
  if (n == 0) return;
  const int blocks = (int)((n + 255) / 256 < 4096 ? (n + 255) / 256 : 4096);
  k_to_f32<<<blocks, 256, 0, st>>>(src, kind, dst, n);
}

__global__ void k_copy_cols(const void* src, int kind, const float* scale, float* dst, int rows, int cols, int ld_dst,
                            int col_off) {
  const size_t n = (size_t)rows * cols;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const int r = (int)(i / cols), c = (int)(i % cols);
    float v = load_src(src, kind, i);
    if (scale) v *= scale[c];
    dst[(size_t)r * ld_dst + col_off + c] = v;
  }
}
void launch_copy_cols(const void* src, int kind, const float* scale, float* dst, int rows, int cols, int ld_dst,
                      int col_off, cudaStream_t st) {
  const size_t n = (size_t)rows * cols;
  const int blocks = (int)((n + 255) / 256 < 8192 ? (n + 255) / 256 : 8192);
  k_copy_cols<<<blocks, 256, 0, st>>>(src, kind, scale, dst, rows, cols, ld_dst, col_off);
}

// Weight [K][N] -> packed out-channel-major swizzled blocks.  One thread per 16-byte chunk
// (8 consecutive k of one out channel): reads are strided by N (one-off cost at create).
__device__ __forceinline__ int pair16_row(int np) {
  const int r = np & 127;
  return (np & ~127) | (32 * ((r & 63) >> 4) + 16 * (r >> 6) + (r & 15));
}
__global__ void k_pack_tiled(const void* src, int kind, __nv_bfloat16* dst, int K, int N, int n_off, int il_group,
                             int il_second, int perm_dh, int pair16) {
  const int KC = K >> 6;
  const size_t chunks = (size_t)N * (K >> 3);
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < chunks; i += (size_t)gridDim.x * blockDim.x) {
    const int n = (int)(i % N);         // consecutive threads -> consecutive n: coalesced source reads
    const int k8 = (int)(i / N);        // chunk index along K
    const int k0 = k8 << 3;
    // optional interleave: groups of il_group channels of two matrices alternate in the packed rows
    int np = il_group ? (n / il_group) * (2 * il_group) + (n % il_group) + (il_second ? il_group : 0)
                      : n_off + (perm_dh ? qkv_channel_to_packed(n, perm_dh) : n);
    if (pair16) np = pair16_row(np);
    const int kc = k0 >> 6, c = (k0 & 63) >> 3;
    const size_t base = (((size_t)(np >> 7) * KC + kc) * 128 + (np & 127)) * 64 + (size_t)((c ^ (np & 7)) << 3);
    __align__(16) __nv_bfloat16 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = __float2bfloat16_rn(load_src(src, kind, (size_t)(k0 + j) * N + n));
    *reinterpret_cast<uint4*>(dst + base) = *reinterpret_cast<const uint4*>(v);
  }
}
void launch_pack_tiled(const void* src, int kind, __nv_bfloat16* dst, int K, int N, int n_off, cudaStream_t st,
                       int il_group, int il_second, int perm_dh, int pair16) {
  const size_t chunks = (size_t)N * (K >> 3);
  const int blocks = (int)((chunks + 255) / 256 < 16384 ? (chunks + 255) / 256 : 16384);
  k_pack_tiled<<<blocks, 256, 0, st>>>(src, kind, dst, K, N, n_off, il_group, il_second, perm_dh, pair16);
}

// e4m3 codes [K][N] -> byte blocks of 128 out channels x 64 k (row order as in k_pack_tiled, no swizzle: the kernel
// that decodes them writes the swizzled bf16 image itself).  One thread per 8 consecutive k of one out channel.
__global__ void k_pack_bytes(const uint8_t* src, uint8_t* dst, int K, int N, int n_off, int il_group, int il_second,
                             int perm_dh, int wide, int pair16) {
  const int KC = wide ? K >> 7 : K >> 6;
  const size_t chunks = (size_t)N * (K >> 3);
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < chunks; i += (size_t)gridDim.x * blockDim.x) {
    const int n = (int)(i % N), k0 = (int)(i / N) << 3;
    int np = il_group ? (n / il_group) * (2 * il_group) + (n % il_group) + (il_second ? il_group : 0)
                      : n_off + (perm_dh ? qkv_channel_to_packed(n, perm_dh) : n);
    if (pair16) np = pair16_row(np);
    __align__(8) uint8_t v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = src[(size_t)(k0 + j) * N + n];
    size_t off;
    if (wide) {
      // 128-byte rows: 16-byte chunk ((k0 % 128) / 16) XOR (row % 8), then the 8-byte half inside it
      const int kc = k0 >> 7, w = k0 & 127, r = np & 127;
      off = (((size_t)(np >> 7) * KC + kc) * 128 + r) * 128 + (size_t)(((w >> 4) ^ (r & 7)) << 4) + (size_t)(w & 8);
    } else {
      const int kc = k0 >> 6, c = (k0 & 63) >> 3;
      off = (((size_t)(np >> 7) * KC + kc) * 128 + (np & 127)) * 64 + (size_t)c * 8;
    }
    *reinterpret_cast<uint2*>(dst + off) = *reinterpret_cast<const uint2*>(v);
  }
}
void launch_pack_bytes(const uint8_t* src, uint8_t* dst, int K, int N, int n_off, cudaStream_t st, int il_group,
                       int il_second, int perm_dh, int wide, int pair16) {
  const size_t chunks = (size_t)N * (K >> 3);
  const int blocks = (int)((chunks + 255) / 256 < 16384 ? (chunks + 255) / 256 : 16384);
  k_pack_bytes<<<blocks, 256, 0, st>>>(src, dst, K, N, n_off, il_group, il_second, perm_dh, wide, pair16);
}

// row-major bf16 [M][K] -> tiled bf16 [K/64][rows_pad][64] (16-byte chunks XOR-swizzled by row & 7)
__global__ void k_rows_to_tiled(const __nv_bfloat16* x, __nv_bfloat16* t, int M, int K, int rows_pad) {
  const size_t n = (size_t)M * (K >> 3);
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const int row = (int)(i / (K >> 3)), c8 = (int)(i % (K >> 3));
    const uint4 v = *reinterpret_cast<const uint4*>(x + (size_t)row * K + c8 * 8);
    *reinterpret_cast<uint4*>(t + tiled_index(row, c8 * 8, rows_pad)) = v;
  }
}
void launch_rows_to_tiled(const __nv_bfloat16* x, __nv_bfloat16* tiled, int M, int K, int rows_pad, cudaStream_t st) {
  const size_t n = (size_t)M * (K >> 3);
  k_rows_to_tiled<<<(int)((n + 255) / 256 < 4096 ? (n + 255) / 256 : 4096), 256, 0, st>>>(x, tiled, M, K, rows_pad);
}

// W8A8 activation quantization: one warp per token row.  A lane takes the 16-column groups lane, lane + 32, ... of
// the row (two 16-byte chunks of the bf16 tile -> one 16-byte chunk of the e4m3 tile); the row stays in registers
// between the maximum and the rounding.  The division by the scale is the IEEE one, so that the rounding decision
// depends on nothing but the stored activations.
constexpr int QR_MAXG = 8;    // 16-column groups per lane: K <= 32 * 8 * 16 = 4096
__global__ void __launch_bounds__(256) k_quant_rows(const int* status, const __nv_bfloat16* x, uint8_t* out, float* scale,
                                                    int rows_pad, int M, int K) {
  pdl_enter();
  if (status_set(status)) return;
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= M) return;
  const int groups = K >> 4;
  uint4 v[QR_MAXG][2];
  float amax = 0.f;
#pragma unroll
  for (int j = 0; j < QR_MAXG; ++j) {
    const int gi = lane + 32 * j;
    if (gi < groups) {
      const int col = gi << 4, kc = col >> 6, c = (col & 63) >> 3;           // two consecutive 8-column chunks c, c + 1
      const __nv_bfloat16* base = x + ((size_t)kc * rows_pad + row) * 64;
      v[j][0] = *reinterpret_cast<const uint4*>(base + ((c ^ (row & 7)) << 3));
      v[j][1] = *reinterpret_cast<const uint4*>(base + (((c + 1) ^ (row & 7)) << 3));
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint32_t w[4] = {v[j][h].x, v[j][h].y, v[j][h].z, v[j][h].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const __nv_bfloat162 p = *reinterpret_cast<const __nv_bfloat162*>(&w[e]);
          amax = fmaxf(amax, fmaxf(fabsf(__low2float(p)), fabsf(__high2float(p))));
        }
      }
    }
  }
  amax = warp_max(amax);
  const float s = amax > 0.f ? __fdiv_rn(amax, 448.0f) : 1.0f;
  if (lane == 0) scale[row] = s;
#pragma unroll
  for (int j = 0; j < QR_MAXG; ++j) {
    const int gi = lane + 32 * j;
    if (gi < groups) {
      uint32_t o[4];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint32_t w[4] = {v[j][h].x, v[j][h].y, v[j][h].z, v[j][h].w};
#pragma unroll
        for (int e = 0; e < 4; e += 2) {
          const __nv_bfloat162 p0 = *reinterpret_cast<const __nv_bfloat162*>(&w[e]);
          const __nv_bfloat162 p1 = *reinterpret_cast<const __nv_bfloat162*>(&w[e + 1]);
          uint16_t lo, hi;    // cvt packs its first source into the upper byte
          asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(__fdiv_rn(__high2float(p0), s)), "f"(__fdiv_rn(__low2float(p0), s)));
          asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(__fdiv_rn(__high2float(p1), s)), "f"(__fdiv_rn(__low2float(p1), s)));
          o[h * 2 + (e >> 1)] = (uint32_t)lo | ((uint32_t)hi << 16);
        }
      }
      const int col = gi << 4, kc = col >> 7, c16 = (col & 127) >> 4;
      *reinterpret_cast<uint4*>(out + ((size_t)kc * rows_pad + row) * 128 + ((c16 ^ (row & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}
void launch_quant_rows(const int* status, const __nv_bfloat16* x, uint8_t* out, float* scale, int rows_pad, int M, int K,
                       cudaStream_t st) {
  launch_pdl(k_quant_rows, dim3((M + 7) / 8), dim3(256), 0, st, status, x, out, scale, rows_pad, M, K);
}

// int4 codes: source [K][N/2] with two neighbouring out channels per byte; destination blocks of 128 out channels x
// 64 k with two neighbouring k per byte (what a row of the MMA's K-major operand needs).  One thread per 8 k of one
// out channel (4 destination bytes).
__global__ void k_pack_nibbles(const uint8_t* src, uint8_t* dst, int K, int N, int n_off, int il_group, int il_second,
                               int perm_dh) {
  const int KC = K >> 6;
  const size_t chunks = (size_t)N * (K >> 3);
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < chunks; i += (size_t)gridDim.x * blockDim.x) {
    const int n = (int)(i % N), k0 = (int)(i / N) << 3;
    const int np = il_group ? (n / il_group) * (2 * il_group) + (n % il_group) + (il_second ? il_group : 0)
                            : n_off + (perm_dh ? qkv_channel_to_packed(n, perm_dh) : n);
    uint32_t w = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint8_t b = src[(size_t)(k0 + j) * (N >> 1) + (n >> 1)];
      const uint32_t c = (n & 1) ? (b >> 4) : (b & 15);
      w |= c << (4 * j);
    }
    const int kc = k0 >> 6;
    *reinterpret_cast<uint32_t*>(dst + (((size_t)(np >> 7) * KC + kc) * 128 + (np & 127)) * 32 + ((k0 & 63) >> 1)) = w;
  }
}
void launch_pack_nibbles(const uint8_t* src, uint8_t* dst, int K, int N, int n_off, cudaStream_t st, int il_group,
                         int il_second, int perm_dh) {
  const size_t chunks = (size_t)N * (K >> 3);
  const int blocks = (int)((chunks + 255) / 256 < 16384 ? (chunks + 255) / 256 : 16384);
  k_pack_nibbles<<<blocks, 256, 0, st>>>(src, dst, K, N, n_off, il_group, il_second, perm_dh);
}

// Row of an adaptive norm's shift through a packed weight matrix: out[n] = scale(n) * sum_k shift[k] * W[n][k].
// One warp per packed row; a lane reads pairs of k out of the swizzled 128 x 64 blocks.
__global__ void k_shift_rows(const float* shift, const __nv_bfloat16* Wp, const float* wscale, const float* wscale2,
                             int interleaved, float* out, int N, int K) {
  const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (n >= N) return;
  const int KC = K >> 6, tile = n >> 7, r = n & 127;
  float acc = 0.f;
  for (int k2 = lane * 2; k2 < K; k2 += 64) {
    const int kc = k2 >> 6, w = k2 & 63, c = w >> 3;
    const size_t idx = (((size_t)tile * KC + kc) * 128 + r) * 64 + (size_t)((c ^ (r & 7)) << 3) + (w & 7);
    const __nv_bfloat162 p = *reinterpret_cast<const __nv_bfloat162*>(Wp + idx);
    acc = fmaf(shift[k2], __low2float(p), acc);
    acc = fmaf(shift[k2 + 1], __high2float(p), acc);
  }
  acc = warp_sum(acc);
  if (lane == 0) {
    float sc = 1.0f;
    if (interleaved) {
      const float* sp = r >= 64 ? wscale2 : wscale;
      if (sp) sc = sp[tile * 64 + (r & 63)];
    } else if (wscale) {
      sc = wscale[n];
    }
    out[n] = acc * sc;
  }
}
void launch_shift_rows(const float* shift, const __nv_bfloat16* Wp, const float* wscale, const float* wscale2,
                       int interleaved, float* out, int N, int K, cudaStream_t st) {
  k_shift_rows<<<(N + 7) / 8, 256, 0, st>>>(shift, Wp, wscale, wscale2, interleaved, out, N, K);
}

// dst[n_off + packed(c)] = src[c]: per-channel scales in the packed row order of the fused QKV matrix
__global__ void k_permute_scales(const float* src, float* dst, int N, int n_off, int perm_dh) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c < N) dst[n_off + (perm_dh ? qkv_channel_to_packed(c, perm_dh) : c)] = src[c];
}
void launch_permute_scales(const float* src, float* dst, int N, int n_off, int perm_dh, cudaStream_t st) {
  k_permute_scales<<<(N + 255) / 256, 256, 0, st>>>(src, dst, N, n_off, perm_dh);
}

// =============================================================================================
// tables
// =============================================================================================
__global__ void k_rows_gemm(const float* X, int ldx, const void* W, int w_kind, int w_row_off, int N, int K,
                            const float* bias, const float* add, int act_swish, float* Y, int ldy) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int r = blockIdx.y;
  if (n >= N) return;
  double acc = 0.0;
  const float* x = X + (size_t)r * ldx;
  for (int d = 0; d < K; ++d) acc += (double)x[d] * (double)load_src(W, w_kind, (size_t)(w_row_off + d) * N + n);
  if (bias) acc += (double)bias[n];
  if (add) acc += (double)add[n];
  if (act_swish) acc = acc / (1.0 + exp(-acc));
  Y[(size_t)r * ldy + n] = (float)acc;
}
void launch_rows_gemm(const float* X, int ldx, const void* W, int w_kind, int w_row_off, int N, int K, const float* bias,
                      const float* add, int act_swish, float* Y, int ldy, int R, cudaStream_t st) {
  dim3 grid((N + 127) / 128, R);
  k_rows_gemm<<<grid, 128, 0, st>>>(X, ldx, W, w_kind, w_row_off, N, K, bias, add, act_swish, Y, ldy);
}

// tau[k][j] = sin(2 pi t_k / period_j), tau[k][D/2 + j] = cos(...), t_k = 1 - k/n, in fp64.
__global__ void k_sinusoid(float* tau, int n_steps, int D, double pmin, double pmax) {
  const int half = D / 2;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_steps * half) return;
  const int k = idx / half, j = idx % half;
  const double t = 1.0 - (double)k / (double)n_steps;
  const double frac = half > 1 ? (double)j / (double)(half - 1) : 0.0;
  const double period = pmin * pow(pmax / pmin, frac);
  const double arg = 6.283185307179586476925286766559 * t / period;
  tau[(size_t)k * D + j] = (float)sin(arg);
  tau[(size_t)k * D + half + j] = (float)cos(arg);
}
void launch_sinusoid(float* tau, int n_steps, int D, double pmin, double pmax, cudaStream_t st) {
  const int n = n_steps * (D / 2);
  k_sinusoid<<<(n + 127) / 128, 128, 0, st>>>(tau, n_steps, D, pmin, pmax);
}

__global__ void k_rope_table(float2* tab, int n_pos, int dh, double theta) {
  const int half = dh / 2;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_pos * half) return;
  const int pos = idx / half, j = idx % half;
  const double phi = (double)pos * pow(theta, -2.0 * (double)j / (double)dh);
  tab[idx] = make_float2((float)cos(phi), (float)sin(phi));
}
void launch_rope_table(float2* tab, int n_pos, int dh, double theta, cudaStream_t st) {
  const int n = n_pos * (dh / 2);
  k_rope_table<<<(n + 127) / 128, 128, 0, st>>>(tab, n_pos, dh, theta);
}

__global__ void k_one_plus(const float* g, float* out, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = 1.0f + g[i];
}
void launch_one_plus(const float* gamma, float* out, int n, cudaStream_t st) {
  k_one_plus<<<(n + 255) / 256, 256, 0, st>>>(gamma, out, n);
}

__global__ void k_mod_finish(float* mod, int R, int D) {
  const size_t n = (size_t)R * D;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const size_t r = i / D, d = i % D;
    mod[r * 3 * D + d] += 1.0f;
  }
}
void launch_mod_finish(float* mod, int R, int D, cudaStream_t st) {
  k_mod_finish<<<256, 256, 0, st>>>(mod, R, D);
}

// =============================================================================================
// per-call prologue: x <- noise, state-token rows
// =============================================================================================
__global__ void k_begin(const Request* rq, const int* status, const float* Ws, const float* bs, float* state_tok,
                        int Ds, int D, int HA, int batch, int ns) {
  if (status_set(status)) return;
  const Request r = *rq;
  const size_t total = (size_t)batch * HA;
  const size_t tid = blockIdx.x * (size_t)blockDim.x + threadIdx.x, nth = (size_t)gridDim.x * blockDim.x;
  if (r.x != r.noise)
    for (size_t i = tid; i < total; i += nth) r.x[i] = r.noise[i];
  if (ns) {
    const size_t tot2 = (size_t)batch * D;
    for (size_t i = tid; i < tot2; i += nth) {
      const int b = (int)(i / D), n = (int)(i % D);
      float acc = 0.f;
      for (int s = 0; s < Ds; ++s) acc = fmaf(r.states[(size_t)b * Ds + s], Ws[(size_t)s * D + n], acc);
      state_tok[i] = acc + bs[n];
    }
  }
}
void launch_begin(const Request* rq, const int* status, const float* Ws, const float* bs, float* state_tok,
                  const Dims& d, int batch, cudaStream_t st) {
  const size_t work = (size_t)batch * (d.H * d.A > d.D ? d.H * d.A : d.D);
  const int blocks = (int)((work + 255) / 256 < 1024 ? (work + 255) / 256 : 1024);
  k_begin<<<blocks, 256, 0, st>>>(rq, status, Ws, bs, state_tok, d.Ds, d.D, d.H * d.A, batch, d.ns);
}

// =============================================================================================
// suffix embedding
// =============================================================================================
// pi0 (time concatenated into the action MLP): with the first MLP layer folded into the action
// projection, u = swish(x Wc + tb_k) where Wc = Wa W1[0:D] and tb_k = tau_k W1[D:2D] + b1 + ba W1[0:D].
template <class Writer>
__global__ void k_embed_pi0(const Request* rq, const int* status, const float* Wc, const float* tb,
                            const float* state_tok, float* h, Writer u, int A, int H, int D, int S, int ns) {
  if (status_set(status)) return;
  extern __shared__ float xs[];
  const int r = blockIdx.x;  // action row b*H + i
  const int b = r / H, i = r % H;
  const float* x = rq->x + (size_t)r * A;
  for (int a = threadIdx.x; a < A; a += blockDim.x) xs[a] = x[a];
  __syncthreads();
  for (int n = threadIdx.x; n < D; n += blockDim.x) {
    float acc = 0.f;
#pragma unroll 8
    for (int a = 0; a < A; ++a) acc = fmaf(xs[a], __ldg(Wc + (size_t)a * D + n), acc);   // loads of 8 rows in flight
    u.store(r, n, swish_precise(acc + tb[n]));
    if (ns && i == 0) h[(size_t)(b * S) * D + n] = state_tok[(size_t)b * D + n];
  }
}
// Tiled-bf16 variant for large batches: one block takes ER action rows, a thread four consecutive output channels
// of all of them, so an element of Wc is fetched once per ER rows and the results leave as 8-byte stores.
constexpr int ER = 16;
__global__ void __launch_bounds__(256) k_embed_pi0_rows(const Request* rq, const int* status, const float* Wc,
                                                        const float* tb, const float* state_tok, float* h,
                                                        __nv_bfloat16* u, int rows_pad, int A, int H, int D, int S, int ns,
                                                        int rows_total) {
  pdl_enter();
  if (status_set(status)) return;
  extern __shared__ float xs[];            // ER x A
  const int r0 = blockIdx.x * ER;
  for (int idx = threadIdx.x; idx < ER * A; idx += blockDim.x) {
    const int r = r0 + idx / A;
    xs[idx] = r < rows_total ? rq->x[(size_t)r * A + idx % A] : 0.f;
  }
  __syncthreads();
  for (int n = threadIdx.x * 4; n < D; n += blockDim.x * 4) {
    float4 acc[ER];
#pragma unroll
    for (int e = 0; e < ER; ++e) acc[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int a = 0; a < A; ++a) {
      const float4 w = __ldg(reinterpret_cast<const float4*>(Wc + (size_t)a * D + n));
#pragma unroll
      for (int e = 0; e < ER; ++e) {
        const float x = xs[e * A + a];
        acc[e].x = fmaf(x, w.x, acc[e].x), acc[e].y = fmaf(x, w.y, acc[e].y);
        acc[e].z = fmaf(x, w.z, acc[e].z), acc[e].w = fmaf(x, w.w, acc[e].w);
      }
    }
    const float4 t4 = __ldg(reinterpret_cast<const float4*>(tb + n));
#pragma unroll
    for (int e = 0; e < ER; ++e) {
      const int r = r0 + e;
      if (r >= rows_total) break;
      __nv_bfloat162 lo = __floats2bfloat162_rn(swish_precise(acc[e].x + t4.x), swish_precise(acc[e].y + t4.y));
      __nv_bfloat162 hi = __floats2bfloat162_rn(swish_precise(acc[e].z + t4.z), swish_precise(acc[e].w + t4.w));
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo), pk.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(u + tiled_index(r, n, rows_pad)) = pk;
      if (ns && r % H == 0)
        *reinterpret_cast<float4*>(h + (size_t)((r / H) * S) * D + n) =
            __ldg(reinterpret_cast<const float4*>(state_tok + (size_t)(r / H) * D + n));
    }
  }
}

void launch_embed_pi0(const Request* rq, const int* status, const float* Wc, const float* tb, const float* state_tok,
                      float* h, float* u_f32, __nv_bfloat16* u_tiled, int rows_pad, const Dims& d, int batch,
                      cudaStream_t st) {
  const int rows = batch * d.H;
  if (u_tiled && d.D % 4 == 0 && rows >= 4 * ER) {
    launch_pdl(k_embed_pi0_rows, dim3((rows + ER - 1) / ER), dim3(256), (size_t)ER * d.A * sizeof(float), st, rq, status,
               Wc, tb, state_tok, h, u_tiled, rows_pad, d.A, d.H, d.D, d.S, d.ns, rows);
    return;
  }
  if (u_tiled)
    k_embed_pi0<<<rows, 256, d.A * sizeof(float), st>>>(rq, status, Wc, tb, state_tok, h, TiledBf16{u_tiled, rows_pad},
                                                        d.A, d.H, d.D, d.S, d.ns);
  else
    k_embed_pi0<<<rows, 256, d.A * sizeof(float), st>>>(rq, status, Wc, tb, state_tok, h, RowMajorF32{u_f32, d.D}, d.A,
                                                        d.H, d.D, d.S, d.ns);
}

__global__ void k_embed_pi05(const Request* rq, const int* status, const float* Wa, const float* ba,
                             const float* state_tok, float* h, int A, int H, int D, int S, int ns) {
  if (status_set(status)) return;
  extern __shared__ float xs[];
  const int r = blockIdx.x;
  const int b = r / H, i = r % H;
  const float* x = rq->x + (size_t)r * A;
  for (int a = threadIdx.x; a < A; a += blockDim.x) xs[a] = x[a];
  __syncthreads();
  float* hrow = h + (size_t)(b * S + ns + i) * D;
  for (int n = threadIdx.x; n < D; n += blockDim.x) {
    float acc = 0.f;
    for (int a = 0; a < A; ++a) acc = fmaf(xs[a], Wa[(size_t)a * D + n], acc);
    hrow[n] = acc + ba[n];
    if (ns && i == 0) h[(size_t)(b * S) * D + n] = state_tok[(size_t)b * D + n];
  }
}
void launch_embed_pi05(const Request* rq, const int* status, const float* Wa, const float* ba, const float* state_tok,
                       float* h, const Dims& d, int batch, cudaStream_t st) {
  k_embed_pi05<<<batch * d.H, 256, d.A * sizeof(float), st>>>(rq, status, Wa, ba, state_tok, h, d.A, d.H, d.D, d.S,
                                                              d.ns);
}

// =============================================================================================
// (Ada)RMSNorm: one warp per row
// =============================================================================================
template <class Writer>
__global__ void k_rmsnorm(const int* status, const float* h, const float* gain, const float* shift, Writer out, int M,
                          int D, float eps) {
  if (status_set(status)) return;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
  const float* x = h + (size_t)row * D;
  float ss = 0.f;
  for (int d = lane; d < D; d += 32) ss = fmaf(x[d], x[d], ss);
  ss = warp_sum(ss);
  const float r = 1.0f / sqrtf(ss / (float)D + eps);
  for (int d = lane; d < D; d += 32) {
    float v = x[d] * r * gain[d];
    if (shift) v += shift[d];
    out.store(row, d, v);
  }
}
// Vectorised variant for the tensor path: D a multiple of 128, tiled bf16 output, one warp per row,
// float4 loads and 8-byte stores.
__global__ void k_rmsnorm_tiled4(const int* status, float* h, const float* gain, const float* shift,
                                 __nv_bfloat16* out, int rows_pad, int M, int D, float eps, SlabSum sl) {
  pdl_enter();
  if (status_set(status)) return;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
  float* x = h + (size_t)row * D;
  float ss = 0.f;
  for (int d = lane * 4; d < D; d += 128) {
    float4 v = *reinterpret_cast<const float4*>(x + d);
    if (sl.n) {   // add the pending split-K partials in slab order and keep the sum (re-read below by this thread)
      for (int s = 0; s < sl.n; ++s) {
        const float4 p = *reinterpret_cast<const float4*>(sl.slab + (size_t)s * sl.stride + (size_t)row * D + d);
        v.x += p.x, v.y += p.y, v.z += p.z, v.w += p.w;
      }
      *reinterpret_cast<float4*>(x + d) = v;
    }
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = warp_sum(ss);
  const float r = 1.0f / sqrtf(ss / (float)D + eps);
  for (int d = lane * 4; d < D; d += 128) {
    const float4 v = *reinterpret_cast<const float4*>(x + d);
    const float4 g = *reinterpret_cast<const float4*>(gain + d);
    float4 o = make_float4(v.x * r * g.x, v.y * r * g.y, v.z * r * g.z, v.w * r * g.w);
    if (shift) {
      const float4 s4 = *reinterpret_cast<const float4*>(shift + d);
      o.x += s4.x, o.y += s4.y, o.z += s4.z, o.w += s4.w;
    }
    __nv_bfloat162 lo = __floats2bfloat162_rn(o.x, o.y), hi = __floats2bfloat162_rn(o.z, o.w);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo), pk.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(out + tiled_index(row, d, rows_pad)) = pk;
  }
}

// Same, with the whole row held in registers (D = NV * 128): every load of the row is in flight at once and the
// row is read once.
// With out8 set (W8A8) the normalised row leaves as its per-token e4m3 quantization instead (codes in the tiled e4m3
// layout, scale in xscale[row]): the bf16 rounding of every element is what gets quantized, as in k_quant_rows.
template <int NV, bool Q8>
__global__ void k_rmsnorm_tiled_reg(const int* status, float* h, const float* gain, const float* shift,
                                    __nv_bfloat16* out, int rows_pad, int M, float eps, SlabSum sl, uint8_t* out8,
                                    float* xscale) {
  pdl_enter();
  if (status_set(status)) return;
  constexpr int D = NV * 128;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
  float* x = h + (size_t)row * D;
  float4 v[NV];
#pragma unroll
  for (int k = 0; k < NV; ++k) v[k] = *reinterpret_cast<const float4*>(x + k * 128 + lane * 4);
  if (sl.n) {   // add the pending split-K partials in slab order and write the row back
    for (int s = 0; s < sl.n; ++s) {
      const float* p = sl.slab + (size_t)s * sl.stride + (size_t)row * D + lane * 4;
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const float4 q = __ldg(reinterpret_cast<const float4*>(p + k * 128));
        v[k].x += q.x, v[k].y += q.y, v[k].z += q.z, v[k].w += q.w;
      }
    }
#pragma unroll
    for (int k = 0; k < NV; ++k) *reinterpret_cast<float4*>(x + k * 128 + lane * 4) = v[k];
  }
  float ss = 0.f;
#pragma unroll
  for (int k = 0; k < NV; ++k) ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
  ss = warp_sum(ss);
  const float r = 1.0f / sqrtf(ss / (float)D + eps);
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    const int d = k * 128 + lane * 4;
    const float4 g = __ldg(reinterpret_cast<const float4*>(gain + d));
    float4 o = make_float4(v[k].x * r * g.x, v[k].y * r * g.y, v[k].z * r * g.z, v[k].w * r * g.w);
    if (shift) {
      const float4 s4 = __ldg(reinterpret_cast<const float4*>(shift + d));
      o.x += s4.x, o.y += s4.y, o.z += s4.z, o.w += s4.w;
    }
    __nv_bfloat162 lo = __floats2bfloat162_rn(o.x, o.y), hi = __floats2bfloat162_rn(o.z, o.w);
    if constexpr (Q8) {   // keep the bf16-rounded values for the quantization below
      v[k] = make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
      continue;
    }
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo), pk.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(out + tiled_index(row, d, rows_pad)) = pk;
  }
  if constexpr (Q8) {
    float amax = 0.f;
#pragma unroll
    for (int k = 0; k < NV; ++k) amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v[k].x), fabsf(v[k].y)), fmaxf(fabsf(v[k].z), fabsf(v[k].w))));
    amax = warp_max(amax);
    const float s = amax > 0.f ? __fdiv_rn(amax, 448.0f) : 1.0f;
    if (lane == 0) xscale[row] = s;
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      uint16_t lo, hi;    // cvt packs its first source into the upper byte
      asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(__fdiv_rn(v[k].y, s)), "f"(__fdiv_rn(v[k].x, s)));
      asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(__fdiv_rn(v[k].w, s)), "f"(__fdiv_rn(v[k].z, s)));
      // channels k * 128 + 4 lane .. + 3: k-chunk k of the e4m3 tile, 16-byte chunk lane / 4, bytes 4 (lane % 4) ..
      *reinterpret_cast<uint32_t*>(out8 + ((size_t)k * rows_pad + row) * 128 + ((((lane >> 2) ^ (row & 7))) << 4) + (lane & 3) * 4) =
          (uint32_t)lo | ((uint32_t)hi << 16);
    }
  }
}

// Row update with pending split-K partials: h[row] += slab_0[row] + slab_1[row] + ... (that order), optionally
// followed by the norm into the tiled bf16 layout.  One block per row, one float4 per thread (D / 4 threads): the
// slab loads of a thread are independent, so they are all in flight together.
__global__ void __launch_bounds__(512) k_add_slabs_norm(const int* status, float* h, const float* gain, const float* shift,
                                                        __nv_bfloat16* out, int rows_pad, int D, float eps, SlabSum sl) {
  // Constants (gain, and the shift row of the modulation table, which is complete before the loop starts) are
  // fetched before the dependency wait; the status word is requested together with the row and its slabs and only
  // looked at once they are summed, so that the three round trips to the L2 overlap.
  pdl_launch_dependents();
  __shared__ float red[16];
  const int row = blockIdx.x, t = threadIdx.x, d = t * 4;
  float4 g = make_float4(0.f, 0.f, 0.f, 0.f), s4 = g;
  if (out) {
    g = __ldg(reinterpret_cast<const float4*>(gain + d));
    if (shift) s4 = __ldg(reinterpret_cast<const float4*>(shift + d));
  }
  pdl_wait();
  float* x = h + (size_t)row * D + d;
  float4 v = *reinterpret_cast<const float4*>(x);
  int stv;
  asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(stv) : "l"(status) : "memory");
  const float* p = sl.slab + (size_t)row * D + d;
#pragma unroll 8
  for (int s = 0; s < sl.n; ++s) {
    const float4 q = __ldg(reinterpret_cast<const float4*>(p + (size_t)s * sl.stride));
    v.x += q.x, v.y += q.y, v.z += q.z, v.w += q.w;
  }
  if (stv != 0) return;
  *reinterpret_cast<float4*>(x) = v;
  if (!out) return;
  float ss = warp_sum(v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w);
  if ((t & 31) == 0) red[t >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += red[w];   // same order in every thread
  const float r = 1.0f / sqrtf(tot / (float)D + eps);
  float4 o = make_float4(v.x * r * g.x, v.y * r * g.y, v.z * r * g.z, v.w * r * g.w);
  if (shift) o.x += s4.x, o.y += s4.y, o.z += s4.z, o.w += s4.w;
  __nv_bfloat162 lo = __floats2bfloat162_rn(o.x, o.y), hi = __floats2bfloat162_rn(o.z, o.w);
  uint2 pk;
  pk.x = *reinterpret_cast<uint32_t*>(&lo), pk.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(out + tiled_index(row, d, rows_pad)) = pk;
}
// h += pending slabs, nothing else (before the velocity head)
void launch_add_slabs(const int* status, float* h, int M, int D, cudaStream_t st, SlabSum sl) {
  if (!sl.n) return;
  launch_pdl(k_add_slabs_norm, dim3(M), dim3(D / 4), 0, st, status, h, (const float*)nullptr, (const float*)nullptr,
             (__nv_bfloat16*)nullptr, 0, D, 0.0f, sl);
}

bool rmsnorm_quantizes(int D) { return D == 1024 || D == 2048; }

void launch_rmsnorm(const int* status, float* h, const float* gain, const float* shift, float* out_f32,
                    __nv_bfloat16* out_tiled, int rows_pad, int M, int D, float eps, cudaStream_t st, SlabSum sl,
                    uint8_t* out8, float* xscale) {
  if (sl.n && !out8 && out_tiled && D % 128 == 0 && D <= 2048) {
    launch_pdl(k_add_slabs_norm, dim3(M), dim3(D / 4), 0, st, status, h, gain, shift, out_tiled, rows_pad, D, eps, sl);
    return;
  }
  // with pending slabs a row costs several times more reads: one warp per block spreads the rows over more SMs
  const int wpb = sl.n ? 1 : 4;
  const int blocks = (M + wpb - 1) / wpb;
  if (out_tiled && D == 1024) {
    if (out8)
      launch_pdl(k_rmsnorm_tiled_reg<8, true>, dim3(blocks), dim3(32 * wpb), 0, st, status, h, gain, shift, out_tiled, rows_pad, M, eps,
                 sl, out8, xscale);
    else
      launch_pdl(k_rmsnorm_tiled_reg<8, false>, dim3(blocks), dim3(32 * wpb), 0, st, status, h, gain, shift, out_tiled, rows_pad, M, eps,
                 sl, out8, xscale);
    return;
  }
  if (out_tiled && D == 2048) {
    if (out8)
      launch_pdl(k_rmsnorm_tiled_reg<16, true>, dim3(blocks), dim3(32 * wpb), 0, st, status, h, gain, shift, out_tiled, rows_pad, M, eps,
                 sl, out8, xscale);
    else
      launch_pdl(k_rmsnorm_tiled_reg<16, false>, dim3(blocks), dim3(32 * wpb), 0, st, status, h, gain, shift, out_tiled, rows_pad, M, eps,
                 sl, out8, xscale);
    return;
  }
  if (out_tiled && D % 128 == 0) {
    launch_pdl(k_rmsnorm_tiled4, dim3(blocks), dim3(32 * wpb), 0, st, status, h, gain, shift, out_tiled, rows_pad, M, D, eps, sl);
    return;
  }
  if (out_tiled)
    k_rmsnorm<<<blocks, 128, 0, st>>>(status, h, gain, shift, TiledBf16{out_tiled, rows_pad}, M, D, eps);
  else
    k_rmsnorm<<<blocks, 128, 0, st>>>(status, h, gain, shift, RowMajorF32{out_f32, D}, M, D, eps);
}

// =============================================================================================
// final norm -> out-projection -> Euler update (epilogue): x += dt * (n . Wout + bout)
// =============================================================================================
// One block normalises FR action rows into shared memory (one warp per two rows).  The contraction over D is
// then split over the 8 warps: warp w takes D/8 consecutive d for all FR rows, lane = action channel, so an
// element of Wout is loaded once per block and used for FR rows, and the normalised rows are read as
// float4.  The 8 partial sums are combined in a fixed order.
template <int FR>
__global__ void __launch_bounds__(256) k_final(const Request* rq, const int* status, const float* h, const float* gain,
                                               const float* shift, const float* Wout, const float* bout, float dt, int A,
                                               int H, int D, int S, int ns, float eps, int rows_total) {
  pdl_enter();
  if (status_set(status)) return;
  extern __shared__ float nrm[];            // FR x D, then 8 x FR x 32 partial sums
  float* part = nrm + (size_t)FR * D;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r0 = blockIdx.x * FR;
  for (int rr = warp; rr < FR; rr += 8) {
    const int r = r0 + rr;
    if (r < rows_total) {
      const int b = r / H, i = r % H;
      const float* x = h + (size_t)(b * S + ns + i) * D;
      float ss = 0.f;
      for (int d = lane; d < D; d += 32) ss = fmaf(x[d], x[d], ss);
      ss = warp_sum(ss);
      const float rs = 1.0f / sqrtf(ss / (float)D + eps);
      for (int d = lane; d < D; d += 32) {
        float v = x[d] * rs * gain[d];
        if (shift) v += shift[d];
        nrm[rr * D + d] = v;
      }
    } else {
      for (int d = lane; d < D; d += 32) nrm[rr * D + d] = 0.f;
    }
  }
  __syncthreads();
  const bool vec = (D & 31) == 0;           // float4 reads of the rows need 8 equal, 4-aligned ranges
  const int dper = vec ? D / 8 : (D + 7) / 8;
  for (int a0 = 0; a0 < A; a0 += 32) {
    const int a = a0 + lane;
    float acc[FR];
#pragma unroll
    for (int rr = 0; rr < FR; ++rr) acc[rr] = 0.f;
    if (a < A && !vec) {
      for (int d = warp * dper; d < min(D, (warp + 1) * dper); ++d) {
        const float w0 = __ldg(Wout + (size_t)d * A + a);
#pragma unroll
        for (int rr = 0; rr < FR; ++rr) acc[rr] = fmaf(nrm[rr * D + d], w0, acc[rr]);
      }
    }
    if (a < A && vec) {
      for (int d = warp * dper; d < (warp + 1) * dper; d += 4) {
        const float w0 = __ldg(Wout + (size_t)d * A + a), w1 = __ldg(Wout + (size_t)(d + 1) * A + a);
        const float w2 = __ldg(Wout + (size_t)(d + 2) * A + a), w3 = __ldg(Wout + (size_t)(d + 3) * A + a);
#pragma unroll
        for (int rr = 0; rr < FR; ++rr) {
          const float4 n4 = *reinterpret_cast<const float4*>(nrm + rr * D + d);
          acc[rr] = fmaf(n4.x, w0, fmaf(n4.y, w1, fmaf(n4.z, w2, fmaf(n4.w, w3, acc[rr]))));
        }
      }
    }
#pragma unroll
    for (int rr = 0; rr < FR; ++rr) part[(warp * FR + rr) * 32 + lane] = acc[rr];
    __syncthreads();
    for (int idx = threadIdx.x; idx < FR * 32; idx += 256) {
      const int rr = idx >> 5, al = idx & 31, r = r0 + rr, aa = a0 + al;
      if (r < rows_total && aa < A) {
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += part[(w * FR + rr) * 32 + al];
        float* xo = rq->x + (size_t)r * A;
        xo[aa] = xo[aa] + dt * (v + bout[aa]);
      }
    }
    __syncthreads();
  }
}
void launch_final(const Request* rq, const int* status, const float* h, const float* gain, const float* shift,
                  const float* Wout, const float* bout, float dt, const Dims& d, int batch, cudaStream_t st) {
  const int rows = batch * d.H;
  static PerDeviceOnce once;
  if (once.needed()) {
    cudaFuncSetAttribute(k_final<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    cudaFuncSetAttribute(k_final<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
    once.done();
  }
  // few rows (one request): two rows per block so that the work spreads over more SMs
  if (rows <= 256)
    launch_pdl(k_final<2>, dim3((rows + 1) / 2), dim3(256), ((size_t)2 * d.D + 8 * 2 * 32) * sizeof(float), st, rq, status, h,
               gain, shift, Wout, bout, dt, d.A, d.H, d.D, d.S, d.ns, d.eps, rows);
  else
    launch_pdl(k_final<16>, dim3((rows + 15) / 16), dim3(256), ((size_t)16 * d.D + 8 * 16 * 32) * sizeof(float), st, rq,
               status, h, gain, shift, Wout, bout, dt, d.A, d.H, d.D, d.S, d.ns, d.eps, rows);
}

// =============================================================================================
// generic fp32 GEMM, 64x64x16 tiles, 256 threads, 4x4 outputs per thread
// =============================================================================================
template <bool DUAL>
__global__ void __launch_bounds__(256) k_simt_gemm(const int* status, SimtGemm g) {
  if (status_set(status)) return;
  __shared__ float As[16][64 + 1];
  __shared__ float Bs[16][64];
  __shared__ float Bs2[DUAL ? 16 : 1][64];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  float acc[4][4] = {}, acc2[4][4] = {};
  for (int k0 = 0; k0 < g.K; k0 += 16) {
    for (int i = threadIdx.x; i < 64 * 16; i += 256) {
      const int m = i >> 4, k = i & 15;
      As[k][m] = (m0 + m < g.M && k0 + k < g.K) ? g.A[(size_t)(m0 + m) * g.lda + k0 + k] : 0.f;
    }
    for (int i = threadIdx.x; i < 16 * 64; i += 256) {
      const int k = i >> 6, n = i & 63;
      const bool ok = (k0 + k < g.K && n0 + n < g.N);
      Bs[k][n] = ok ? g.B[(size_t)(k0 + k) * g.N + n0 + n] : 0.f;
      if (DUAL) Bs2[k][n] = ok ? g.B2[(size_t)(k0 + k) * g.N + n0 + n] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      float a[4], b[4], b2[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        b[j] = Bs[k][tx * 4 + j];
        if (DUAL) b2[j] = Bs2[k][tx * 4 + j];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
          if (DUAL) acc2[i][j] = fmaf(a[i], b2[j], acc2[i][j]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= g.M) continue;
    const int orow = (m / g.rows_in) * g.rows_out + g.row_off + m % g.rows_in;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= g.N) continue;
      float* o = g.out + (size_t)orow * g.ldo + n;
      float v = acc[i][j];
      if (g.epi == EPI_STORE) {
        *o = v + (g.bias ? g.bias[n] : 0.f);
      } else if (g.epi == EPI_SWISH) {
        *o = swish_precise(v + (g.bias ? g.bias[n] : 0.f));
      } else if (g.epi == EPI_RESID) {
        *o = *o + (g.gate ? g.gate[n] * v : v);
      } else {
        *o = gelu_f(v, g.gelu_exact) * acc2[i][j];
      }
    }
  }
}
void launch_simt_gemm(const int* status, const SimtGemm& g, cudaStream_t st) {
  dim3 grid((g.N + 63) / 64, (g.M + 63) / 64);
  if (g.epi == EPI_GEGLU)
    k_simt_gemm<true><<<grid, 256, 0, st>>>(status, g);
  else
    k_simt_gemm<false><<<grid, 256, 0, st>>>(status, g);
}

// =============================================================================================
// generic fp32 attention: one block (4 warps) per (suffix row, query head); every warp walks a
// strided share of the keys with an online softmax; the four partial states merge in shared memory.
// =============================================================================================
template <typename KV, class Writer>
__global__ void __launch_bounds__(128) k_attention_simt(const Request* rq, const int* status, const float* qkv,
                                                        const float2* rope, int layer, Writer out, Dims d) {
  if (status_set(status)) return;
  constexpr int MAXR = 8;  // head_dim <= 256
  extern __shared__ float sm[];
  float* qs = sm;                 // [dh] rotated, pre-scaled query
  float* part = sm + d.dh;        // [4][dh + 2] partial (acc, m, l)
  const int row = blockIdx.x;     // b*S + i
  const int a = blockIdx.y;       // query head
  const int b = row / d.S, i = row % d.S;
  const int hk = a / (d.Hq / d.Hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const Request r = *rq;
  const int p0 = r.cu_lens[b], P = r.cu_lens[b + 1] - p0;
  const int half = d.dh >> 1;
  const float scale = rsqrtf((float)d.dh);
  const bool use_rope = rope != nullptr;

  // query, rotated at position P + i
  const float* qrow = qkv + (size_t)row * d.Nqkv + a * d.dh;
  for (int t = threadIdx.x; t < d.dh; t += blockDim.x) {
    float v = qrow[t];
    if (use_rope) {
      const int j = t < half ? t : t - half;
      const float2 cs = rope[(size_t)(P + i) * half + j];
      const float other = qrow[t < half ? t + half : t - half];
      v = t < half ? v * cs.x - other * cs.y : v * cs.x + other * cs.y;
    }
    qs[t] = v * scale;
  }
  __syncthreads();

  const KV* Kp = reinterpret_cast<const KV*>(r.prefix_kv) + ((size_t)(layer * 2 + 0) * r.kv_tokens + p0) * d.Hkv * d.dh +
                 (size_t)hk * d.dh;
  const KV* Vp = reinterpret_cast<const KV*>(r.prefix_kv) + ((size_t)(layer * 2 + 1) * r.kv_tokens + p0) * d.Hkv * d.dh +
                 (size_t)hk * d.dh;
  const size_t kv_stride = (size_t)d.Hkv * d.dh;

  float m = -INFINITY, l = 0.f, acc[MAXR];
#pragma unroll
  for (int t = 0; t < MAXR; ++t) acc[t] = 0.f;

  const int nkeys = P + d.S;
  for (int j = warp; j < nkeys; j += 4) {
    float dot = 0.f;
    float vreg[MAXR];
    if (j < P) {
      const KV* k = Kp + (size_t)j * kv_stride;
      const KV* v = Vp + (size_t)j * kv_stride;
#pragma unroll
      for (int t = 0; t < MAXR; ++t) {
        const int dd = lane + 32 * t;
        if (dd < d.dh) {
          dot = fmaf(qs[dd], to_float<KV>(k[dd]), dot);
          vreg[t] = to_float<KV>(v[dd]);
        } else {
          vreg[t] = 0.f;
        }
      }
    } else {
      const int js = j - P;
      if (d.block_causal && d.ns && i == 0 && js != 0) continue;  // state token sees only itself (warp-uniform)
      const float* krow = qkv + (size_t)(b * d.S + js) * d.Nqkv + d.Nq + hk * d.dh;
      const float* vrow = krow + d.Hkv * d.dh;
#pragma unroll
      for (int t = 0; t < MAXR; ++t) {
        const int dd = lane + 32 * t;
        if (dd < d.dh) {
          float kvv = krow[dd];
          if (use_rope) {
            const int jj = dd < half ? dd : dd - half;
            const float2 cs = rope[(size_t)(P + js) * half + jj];
            const float other = krow[dd < half ? dd + half : dd - half];
            kvv = dd < half ? kvv * cs.x - other * cs.y : kvv * cs.x + other * cs.y;
          }
          dot = fmaf(qs[dd], kvv, dot);
          vreg[t] = vrow[dd];
        } else {
          vreg[t] = 0.f;
        }
      }
    }
    dot = warp_sum(dot);
    const float mn = fmaxf(m, dot);
    const float corr = __expf(m - mn), p = __expf(dot - mn);
    l = l * corr + p;
#pragma unroll
    for (int t = 0; t < MAXR; ++t) acc[t] = acc[t] * corr + p * vreg[t];
    m = mn;
  }
  float* mine = part + warp * (d.dh + 2);
#pragma unroll
  for (int t = 0; t < MAXR; ++t) {
    const int dd = lane + 32 * t;
    if (dd < d.dh) mine[dd] = acc[t];
  }
  if (lane == 0) {
    mine[d.dh] = m;
    mine[d.dh + 1] = l;
  }
  __syncthreads();
  float mm = -INFINITY;
  for (int w = 0; w < 4; ++w) mm = fmaxf(mm, part[w * (d.dh + 2) + d.dh]);
  float ll = 0.f;
  float wgt[4];
  for (int w = 0; w < 4; ++w) {
    const float mw = part[w * (d.dh + 2) + d.dh];
    wgt[w] = (mw == -INFINITY) ? 0.f : __expf(mw - mm);
    ll += wgt[w] * part[w * (d.dh + 2) + d.dh + 1];
  }
  const float inv = 1.0f / ll;
  for (int t = threadIdx.x; t < d.dh; t += blockDim.x) {
    float o = 0.f;
    for (int w = 0; w < 4; ++w) o += wgt[w] * part[w * (d.dh + 2) + t];
    out.store(row, a * d.dh + t, o * inv);
  }
}

void launch_attention_simt(const Request* rq, const int* status, const float* qkv, const float2* rope, int layer,
                           int kv_is_bf16, float* out_f32, __nv_bfloat16* out_tiled, int rows_pad, const Dims& d,
                           int batch, cudaStream_t st) {
  dim3 grid(batch * d.S, d.Hq);
  const size_t smem = (size_t)(d.dh + 4 * (d.dh + 2)) * sizeof(float);
  if (kv_is_bf16) {
    if (out_tiled)
      k_attention_simt<__nv_bfloat16><<<grid, 128, smem, st>>>(rq, status, qkv, rope, layer,
                                                               TiledBf16{out_tiled, rows_pad}, d);
    else
      k_attention_simt<__nv_bfloat16><<<grid, 128, smem, st>>>(rq, status, qkv, rope, layer,
                                                               RowMajorF32{out_f32, d.Nq}, d);
  } else {
    if (out_tiled)
      k_attention_simt<float><<<grid, 128, smem, st>>>(rq, status, qkv, rope, layer, TiledBf16{out_tiled, rows_pad}, d);
    else
      k_attention_simt<float><<<grid, 128, smem, st>>>(rq, status, qkv, rope, layer, RowMajorF32{out_f32, d.Nq}, d);
  }
}

}  // namespace phyai
