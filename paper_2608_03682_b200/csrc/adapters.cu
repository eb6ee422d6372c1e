// The two small steps either side of the denoising loop that belong to the model adapter (paper, Sec. "Architecture":
// the adapter owns preprocessing, cache layout and action conversion): packing a backbone's padded per-layer K / V
// into the library's ragged prefix-KV layout, and converting the raw action chunk (x at t = 0) into robot actions.
// Both are pure data movement / element-wise work: coalesced 16-byte copies, one thread per output element.
#include <cstdio>
#include <new>

#include "../../include/phyai.h"
#include "kernels.h"

namespace phyai {
namespace {

thread_local char g_ad_err[256] = "";

// cu[0] = 0, cu[b + 1] = cu[b] + lens[b]; a length outside 0..p_max or a total beyond kv_tokens raises the status word
// (INVALID_ARG) and the pack kernel then copies nothing.
__global__ void k_kv_scan(const int* lens, int batch, int p_max, unsigned long long kv_tokens, int* cu, int* status) {
  if (threadIdx.x != 0) return;
  long long acc = 0;
  bool bad = false;
  cu[0] = 0;
  for (int b = 0; b < batch; ++b) {
    const int n = lens[b];
    if (n < 0 || n > p_max) bad = true;
    acc += n < 0 ? 0 : n;
    cu[b + 1] = (int)(acc > 0x7fffffffLL ? 0x7fffffffLL : acc);
  }
  if ((unsigned long long)acc > kv_tokens) bad = true;
  if (bad) atomicExch(status, ST_INVALID_ARG);
}

// src [L][B][p_max][row_bytes], dst [L][2][kv_tokens][row_bytes]: plane (l, kv) of request b, rows p < lens[b], go to
// rows cu[b] + p.  One thread per 16 bytes; grid.y = layer * 2 + (0 = K, 1 = V).
__global__ void k_kv_pack(const uint4* k, const uint4* v, const int* lens, const int* cu, const int* status, uint4* dst,
                          int batch, int p_max, unsigned long long kv_tokens, int row_chunks) {
  if (status_set(status)) return;
  const int layer = blockIdx.y >> 1, is_v = blockIdx.y & 1;
  const uint4* src = (is_v ? v : k) + (size_t)layer * batch * p_max * row_chunks;
  uint4* out = dst + ((size_t)layer * 2 + is_v) * kv_tokens * row_chunks;
  const size_t total = (size_t)batch * p_max * row_chunks;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int c = (int)(i % row_chunks);
    const size_t row = i / row_chunks;
    const int p = (int)(row % p_max), b = (int)(row / p_max);
    if (p < lens[b]) out[((size_t)cu[b] + p) * row_chunks + c] = src[i];
  }
}

// out[b][h][a] = (clip(x[b][h][a]) + 1) / 2 * (q99[a] - q01[a]) + q01[a] for h < H_out, a < A_out
__global__ void k_postprocess(const float* x, const float* q01, const float* q99, float* out, int batch, int H, int A,
                              int H_out, int A_out, float lo, float hi, int do_clip) {
  const size_t total = (size_t)batch * H_out * A_out;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int a = (int)(i % A_out), hh = (int)((i / A_out) % H_out), b = (int)(i / ((size_t)A_out * H_out));
    float v = x[((size_t)b * H + hh) * A + a];
    if (do_clip) v = fminf(fmaxf(v, lo), hi);
    const float lo_q = q01 ? q01[a] : -1.0f, hi_q = q99 ? q99[a] : 1.0f;
    out[i] = (v + 1.0f) * 0.5f * (hi_q - lo_q) + lo_q;
  }
}


// fp32 [tokens][2 * nkv] (K channels, then V channels) -> bf16 rows of the K plane and the V plane of one layer
__global__ void k_kv_planes(const float* src, __nv_bfloat16* kplane, __nv_bfloat16* vplane, int tokens, int nkv) {
  const size_t n = (size_t)tokens * (nkv >> 2) * 2;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const int per_row = (nkv >> 2) * 2;
    const int t = (int)(i / per_row), c4 = (int)(i % per_row);
    const float4 v = *reinterpret_cast<const float4*>(src + (size_t)t * 2 * nkv + c4 * 4);
    const int col = c4 * 4;
    __nv_bfloat16* dst = col < nkv ? kplane + (size_t)t * nkv + col : vplane + (size_t)t * nkv + (col - nkv);
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo), pk.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(dst) = pk;
  }
}

}  // namespace
}  // namespace phyai

extern "C" {

const char* phyai_adapter_last_error(void) { return phyai::g_ad_err; }

phyai_status_t phyai_pack_prefix_kv(const phyai_kv_pack_desc_t* desc, const void* k, const void* v, const int32_t* lens,
                                    void* prefix_kv, uint64_t kv_tokens, int32_t* cu_prefix_lens, int32_t* status_word,
                                    void* stream) {
  using namespace phyai;
  auto bad = [](const char* m) {
    snprintf(g_ad_err, sizeof(g_ad_err), "%s", m);
    return PHYAI_ERR_INVALID_ARG;
  };
  if (!desc || desc->struct_size != sizeof(phyai_kv_pack_desc_t)) return bad("desc is NULL or has a wrong struct_size");
  if (!k || !v || !lens || !prefix_kv || !cu_prefix_lens || !status_word) return bad("a pointer argument is NULL");
  if (!desc->n_layers || !desc->n_kv_heads || !desc->head_dim || !desc->batch || !desc->p_max)
    return bad("a size in desc is zero");
  if (desc->elem_bytes != 2 && desc->elem_bytes != 4) return bad("elem_bytes must be 2 (bfloat16) or 4 (float32)");
  const size_t row_bytes = (size_t)desc->n_kv_heads * desc->head_dim * desc->elem_bytes;
  if (row_bytes % 16) return bad("n_kv_heads * head_dim * elem_bytes must be a multiple of 16");
  if ((reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(prefix_kv)) & 15u)
    return bad("k, v and prefix_kv must be 16-byte aligned");
  if (kv_tokens > 0x7fffffffull || desc->batch > 65535u || desc->n_layers > 32767u) return bad("kv_tokens, batch or n_layers too large");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int chunks = (int)(row_bytes / 16);
  k_kv_scan<<<1, 32, 0, st>>>(lens, (int)desc->batch, (int)desc->p_max, kv_tokens, cu_prefix_lens, status_word);
  const size_t total = (size_t)desc->batch * desc->p_max * chunks;
  const int blocks = (int)((total + 255) / 256 < 2048 ? (total + 255) / 256 : 2048);
  k_kv_pack<<<dim3(blocks, desc->n_layers * 2), 256, 0, st>>>(reinterpret_cast<const uint4*>(k), reinterpret_cast<const uint4*>(v), lens,
                                                             cu_prefix_lens, status_word, reinterpret_cast<uint4*>(prefix_kv),
                                                             (int)desc->batch, (int)desc->p_max, kv_tokens, chunks);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    snprintf(g_ad_err, sizeof(g_ad_err), "kernel launch failed: %s", cudaGetErrorString(e));
    return PHYAI_ERR_CUDA;
  }
  return PHYAI_OK;
}

phyai_status_t phyai_postprocess_actions(const float* x, uint32_t batch, uint32_t horizon, uint32_t action_dim,
                                         const float* q01, const float* q99, float clip_lo, float clip_hi,
                                         uint32_t out_horizon, uint32_t out_dim, float* out, void* stream) {
  using namespace phyai;
  if (!x || !out || !batch || !horizon || !action_dim || !out_horizon || !out_dim || out_horizon > horizon ||
      out_dim > action_dim || ((q01 == nullptr) != (q99 == nullptr))) {
    snprintf(g_ad_err, sizeof(g_ad_err), "NULL pointer, zero size, out_horizon > horizon, out_dim > action_dim, or only one of q01 / q99 given");
    return PHYAI_ERR_INVALID_ARG;
  }
  const size_t total = (size_t)batch * out_horizon * out_dim;
  const int blocks = (int)((total + 255) / 256 < 1024 ? (total + 255) / 256 : 1024);
  k_postprocess<<<blocks, 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(x, q01, q99, out, (int)batch, (int)horizon,
                                                                           (int)action_dim, (int)out_horizon, (int)out_dim,
                                                                           clip_lo, clip_hi, clip_lo < clip_hi ? 1 : 0);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    snprintf(g_ad_err, sizeof(g_ad_err), "kernel launch failed: %s", cudaGetErrorString(e));
    return PHYAI_ERR_CUDA;
  }
  return PHYAI_OK;
}

}  // extern "C"

// Request-local K / V projections of a feature-handoff head: per layer one tcgen05 GEMM of the (tiled) feature rows
// against [Wk | Wv], fp32 out, then the bf16 rows of the two planes.  The projector handle owns the packed weight
// images and the workspace, so that a run only enqueues kernels.
struct phyai_kv_projector {
  int L = 0, nkv = 0, Dv = 0, max_tokens = 0, rows_pad = 0;
  __nv_bfloat16* wp = nullptr;    // [L] packed [Wk | Wv] images, Dv x 2 nkv each
  __nv_bfloat16* xt = nullptr;    // tiled features [Dv / 64][rows_pad][64]
  float* y = nullptr;             // [max_tokens][2 nkv]
  int* status = nullptr;
};

namespace {
phyai_status_t proj_fail(phyai_status_t st, const char* msg, cudaError_t e = cudaSuccess) {
  using namespace phyai;
  if (e != cudaSuccess) snprintf(g_ad_err, sizeof(g_ad_err), "%s: %s", msg, cudaGetErrorString(e));
  else snprintf(g_ad_err, sizeof(g_ad_err), "%s", msg);
  return st;
}
}  // namespace

extern "C" void phyai_kv_projector_destroy(phyai_kv_projector_t* p) {
  if (!p) return;
  cudaFree(p->wp), cudaFree(p->xt), cudaFree(p->y), cudaFree(p->status);
  delete p;
}

extern "C" phyai_status_t phyai_kv_projector_create(const phyai_kv_proj_desc_t* desc, const void* const* wk,
                                                    const void* const* wv, uint64_t max_tokens, void* stream,
                                                    phyai_kv_projector_t** out) {
  using namespace phyai;
  g_ad_err[0] = 0;
  if (out) *out = nullptr;
  if (!desc || desc->struct_size != sizeof(phyai_kv_proj_desc_t) || !wk || !wv || !out)
    return proj_fail(PHYAI_ERR_INVALID_ARG, "NULL argument or wrong struct_size");
  const int L = (int)desc->n_layers, nkv = (int)(desc->n_kv_heads * desc->head_dim), Dv = (int)desc->feat_dim;
  if (L <= 0 || nkv <= 0 || Dv <= 0 || Dv % 64 || (2 * nkv) % 128 || max_tokens == 0 || max_tokens > (1u << 22))
    return proj_fail(PHYAI_ERR_INVALID_ARG,
                     "need feat_dim a multiple of 64, 2 * n_kv_heads * head_dim a multiple of 128, 1 <= max_tokens <= 2^22");
  for (int l = 0; l < L; ++l)
    if (!wk[l] || !wv[l]) return proj_fail(PHYAI_ERR_INVALID_ARG, "a per-layer weight pointer is NULL");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  cudaError_t e = tc_gemm_setup();
  if (e != cudaSuccess) return proj_fail(PHYAI_ERR_CUDA, "tc_gemm_setup", e);
  phyai_kv_projector* p = new (std::nothrow) phyai_kv_projector();
  if (!p) return proj_fail(PHYAI_ERR_OOM, "host allocation failed");
  p->L = L, p->nkv = nkv, p->Dv = Dv, p->max_tokens = (int)max_tokens, p->rows_pad = ((int)max_tokens + 255) / 256 * 256;
  const size_t N = 2 * (size_t)nkv;
  if ((e = cudaMalloc(&p->wp, (size_t)L * Dv * N * 2)) != cudaSuccess || (e = cudaMalloc(&p->xt, (size_t)p->rows_pad * Dv * 2)) != cudaSuccess ||
      (e = cudaMalloc(&p->y, (size_t)max_tokens * N * 4)) != cudaSuccess || (e = cudaMalloc(&p->status, 4)) != cudaSuccess) {
    phyai_kv_projector_destroy(p);
    return proj_fail(PHYAI_ERR_OOM, "cudaMalloc", e);
  }
  cudaMemsetAsync(p->xt, 0, (size_t)p->rows_pad * Dv * 2, st);
  cudaMemsetAsync(p->status, 0, 4, st);
  for (int l = 0; l < L; ++l) {
    launch_pack_tiled(wk[l], 1, p->wp + (size_t)l * Dv * N, Dv, nkv, 0, st);
    launch_pack_tiled(wv[l], 1, p->wp + (size_t)l * Dv * N, Dv, nkv, nkv, st);
  }
  e = cudaStreamSynchronize(st);
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) {
    phyai_kv_projector_destroy(p);
    return proj_fail(PHYAI_ERR_CUDA, "weight packing", e);
  }
  *out = p;
  return PHYAI_OK;
}

extern "C" phyai_status_t phyai_kv_projector_run(phyai_kv_projector_t* p, const void* features, uint64_t tokens,
                                                 uint64_t kv_tokens, void* prefix_kv, void* stream) {
  using namespace phyai;
  g_ad_err[0] = 0;
  if (!p || !features || !prefix_kv) return proj_fail(PHYAI_ERR_INVALID_ARG, "NULL argument");
  if (tokens == 0 || tokens > (uint64_t)p->max_tokens || tokens > kv_tokens)
    return proj_fail(PHYAI_ERR_INVALID_ARG, "need 1 <= tokens <= max_tokens and tokens <= kv_tokens");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int M = (int)tokens, N = 2 * p->nkv;
  launch_rows_to_tiled(reinterpret_cast<const __nv_bfloat16*>(features), p->xt, M, p->Dv, p->rows_pad, st);
  __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(prefix_kv);
  for (int l = 0; l < p->L; ++l) {
    TcGemm g{};
    g.W = p->wp + (size_t)l * p->Dv * N, g.X = p->xt, g.M = M, g.N = N, g.K = p->Dv, g.epi = TC_STORE, g.out_f32 = p->y, g.ldo = N;
    g.splits = 1, g.rows_pad = p->rows_pad, g.wait_limit = 1u << 28;
    cudaError_t e = launch_tc_gemm(p->status, g, M <= 64 ? 64 : (M <= 1024 ? 128 : 256), st);
    if (e != cudaSuccess) return proj_fail(PHYAI_ERR_CUDA, "projection GEMM launch", e);
    const size_t n = (size_t)M * (p->nkv >> 2) * 2;
    k_kv_planes<<<(int)((n + 255) / 256 < 4096 ? (n + 255) / 256 : 4096), 256, 0, st>>>(
        p->y, out + ((size_t)l * 2) * kv_tokens * p->nkv, out + ((size_t)l * 2 + 1) * kv_tokens * p->nkv, M, p->nkv);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return proj_fail(PHYAI_ERR_CUDA, "kernel launch failed", e);
  return PHYAI_OK;
}

// One-shot form: create, run, synchronise, destroy.
extern "C" phyai_status_t phyai_project_features_kv(const phyai_kv_proj_desc_t* desc, const void* features,
                                                    const void* const* wk, const void* const* wv, uint64_t tokens,
                                                    uint64_t kv_tokens, void* prefix_kv, void* stream) {
  phyai_kv_projector_t* p = nullptr;
  phyai_status_t st = phyai_kv_projector_create(desc, wk, wv, tokens ? tokens : 1, stream, &p);
  if (st != PHYAI_OK) return st;
  st = phyai_kv_projector_run(p, features, tokens, kv_tokens, prefix_kv, stream);
  cudaError_t e = cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream));
  int hs = 0;
  if (e == cudaSuccess) e = cudaMemcpy(&hs, p->status, 4, cudaMemcpyDeviceToHost);
  phyai_kv_projector_destroy(p);
  if (st != PHYAI_OK) return st;
  if (e != cudaSuccess) return proj_fail(PHYAI_ERR_CUDA, "feature K/V projection", e);
  if (hs != 0) return proj_fail(PHYAI_ERR_TIMEOUT, "a bounded device-side wait expired");
  return PHYAI_OK;
}
