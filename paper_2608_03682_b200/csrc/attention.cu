// Suffix -> (prefix U suffix) attention on tensor cores (operator-selection paragraph of the paper:
// a ~50-token query against a longer prefix with head dimension 256).
//
// Few queries, long shared KV: one CTA takes the (<= 64) suffix rows of HPC query heads that share a
// kv head and a contiguous slice of that request's keys.  K/V tiles are staged into shared memory
// with 16-byte asynchronous copies issued by all threads into XOR-swizzled rows (bank-conflict-free
// ldmatrix), double buffered.  (Per-row bulk copies were measured first: one warp's bulk copies
// complete one at a time, which made 128 small copies per tile the bottleneck.)  Q K^T and P V run on
// mma.sync m16n8k16 (bf16 in,
// fp32 out); the softmax is the online form in fp32 with quad shuffles for the row max / sum.
// The suffix's own K/V (fp32 from the QKV GEMM) are rotated and appended as the last tile.
// When the key range is split over several CTAs each writes an unnormalised partial (O, m, l) and a
// merge kernel combines them.
#include <cstdio>
#include <mutex>

#include "../../include/phyai.h"
#include "kernels.h"
#include "ptx.cuh"
#include "attention.cuh"

namespace phyai {
namespace {

// Combine the per-split partials: out = sum_s 2^(m_s - m) O_s / sum_s 2^(m_s - m) l_s.
template <int DH>
__global__ void k_attn_merge(const int* status, const float* part_o, const float* part_ml, __nv_bfloat16* out,
                             int rows_pad, int num_splits, int S, int Hq) {
  pdl_enter();
  if (status_set(status)) return;
  const int row = blockIdx.x, head = blockIdx.y, b = blockIdx.z;
  const size_t slab0 = ((size_t)(b * Hq + head) * num_splits) * QROWS;
  float mm = -INFINITY;
  for (int s = 0; s < num_splits; ++s) mm = fmaxf(mm, part_ml[(slab0 + (size_t)s * QROWS + row) * 2]);
  float ll = 0.f;
  for (int s = 0; s < num_splits; ++s) {
    const float* ml = part_ml + (slab0 + (size_t)s * QROWS + row) * 2;
    if (ml[0] != -INFINITY) ll += exp2f(ml[0] - mm) * ml[1];
  }
  const float inv = 1.0f / ll;
  for (int c = threadIdx.x * 2; c < DH; c += blockDim.x * 2) {
    float a0 = 0.f, a1 = 0.f;
    for (int s = 0; s < num_splits; ++s) {
      const float ms = part_ml[(slab0 + (size_t)s * QROWS + row) * 2];
      if (ms == -INFINITY) continue;
      const float w = exp2f(ms - mm);
      const float2 v = *reinterpret_cast<const float2*>(part_o + (slab0 + (size_t)s * QROWS + row) * DH + c);
      a0 = fmaf(w, v.x, a0), a1 = fmaf(w, v.y, a1);
    }
    *reinterpret_cast<uint32_t*>(out + out_index(b * S + row, head * DH + c, rows_pad, Hq * DH)) =
        pack_bf16(a0 * inv, a1 * inv);
  }
}

template <int DH, int HPC, int KTT>
constexpr size_t attn_smem() {
  return (size_t)(HPC * QROWS + 4 * KTT) * DH * 2;
}

template <int DH, int HPC, int KTT>
cudaError_t launch_attn(const AttnArgs& a, int batch, cudaStream_t st) {
  static PerDeviceOnce once;
  if (once.needed()) {
    cudaError_t e = cudaFuncSetAttribute(k_attn_mma<DH, HPC, KTT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)attn_smem<DH, HPC, KTT>());
    if (e != cudaSuccess) return e;
    once.done();
  }
  dim3 grid(a.num_splits, a.d.Hq / HPC, batch);
  cudaError_t e = launch_pdl(k_attn_mma<DH, HPC, KTT>, grid, dim3(HPC * 128), attn_smem<DH, HPC, KTT>(), st, a);
  if (e == cudaSuccess && a.num_splits > 1) {
    dim3 g2(a.d.S, a.d.Hq, batch);
    e = launch_pdl(k_attn_merge<DH>, g2, dim3(128), 0, st, a.status, a.part_o, a.part_ml, a.out, a.rows_pad, a.num_splits,
                   a.d.S, a.d.Hq);
  }
  return e;
}

template <int DH, int KTT>
constexpr size_t attn_cluster_smem() {   // Q / K / V buffers + the receive area of the push merge
  return attn_smem<DH, 1, KTT>() + (size_t)8 * 8 * (DH + 4) * 4 + 512;
}

template <int DH, int KTT, bool OPROJ = false>
cudaError_t launch_attn_cluster(const AttnArgs& a, int batch, cudaStream_t st) {
  static PerDeviceOnce once;
  const size_t smem = attn_cluster_smem<DH, KTT>() + (OPROJ ? 1024 : 0);
  if (once.needed()) {
    cudaError_t e = cudaFuncSetAttribute(k_attn_cluster<DH, KTT, OPROJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    once.done();
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(8, a.d.Hq, batch), cfg.blockDim = dim3(128), cfg.dynamicSmemBytes = smem, cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 8, at[0].val.clusterDim.y = 1, at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at, cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, k_attn_cluster<DH, KTT, OPROJ>, a);
}

}  // namespace

// Key-split attention whose partials are merged through distributed shared memory (clusters of 8 CTAs).
// With `op` set, the output projection of each head follows in the same kernel (see attention_oproj_supported).
cudaError_t launch_attention_cluster(const Request* rq, int* status, const float* qkv, const float2* rope,
                                     const __nv_bfloat16* qr, const __nv_bfloat16* kr, const __nv_bfloat16* vr, int layer,
                                     __nv_bfloat16* out_tiled, int rows_pad, const Dims& d, int batch, unsigned wait_limit,
                                     cudaStream_t st, const AttnOproj* op, unsigned long long* trace) {
  AttnArgs a{};
  a.trace = trace;
  a.rq = rq, a.status = status, a.qkv = qkv, a.rope = rope, a.layer = layer, a.out = out_tiled, a.rows_pad = rows_pad;
  a.qr = qr, a.kr = kr, a.vr = vr;   // when set: rotated bf16 operands instead of the fp32 QKV output
  a.num_splits = 8, a.d = d, a.wait_limit = wait_limit;
  if (op) {
    a.wo = op->wo, a.o_scale = op->scale, a.o_gate = op->gate, a.slab = op->slab, a.slab_stride = op->slab_stride, a.D = d.D;
    return launch_attn_cluster<256, 64, true>(a, batch, st);
  }
  if (d.dh == 256) return launch_attn_cluster<256, 64>(a, batch, st);
  if (d.dh == 128) return launch_attn_cluster<128, 64>(a, batch, st);
  return launch_attn_cluster<64, 64>(a, batch, st);
}
// The fused projection covers: head_dim 256, 8 out-channel tiles of 128 (one per CTA of the cluster), a suffix of at
// most 56 rows (the activation tile is packed at 56 rows per k-chunk), rotated bf16 operands.
bool attention_oproj_supported(const Dims& d) { return d.dh == 256 && d.D == 1024 && d.S <= 56 && d.Hq <= 16; }

bool attention_mma_supported(const Dims& d) {
  return (d.dh == 64 || d.dh == 128 || d.dh == 256) && d.S <= QROWS;
}

cudaError_t launch_attention_merge(int* status, const float* part_o, const float* part_ml, __nv_bfloat16* out, int rows_pad,
                                   int num_splits, const Dims& d, int batch, cudaStream_t st) {
  dim3 g2(d.S, d.Hq, batch);
  if (d.dh == 256) return launch_pdl(k_attn_merge<256>, g2, dim3(128), 0, st, status, part_o, part_ml, out, rows_pad, num_splits, d.S, d.Hq);
  if (d.dh == 128) return launch_pdl(k_attn_merge<128>, g2, dim3(128), 0, st, status, part_o, part_ml, out, rows_pad, num_splits, d.S, d.Hq);
  return launch_pdl(k_attn_merge<64>, g2, dim3(128), 0, st, status, part_o, part_ml, out, rows_pad, num_splits, d.S, d.Hq);
}

int attention_pick_splits(const Dims& d, int batch, int max_prefix) {
  const int ctas = batch * d.Hq;
  int want = (2 * 148 + ctas - 1) / ctas;
  const int tiles = (max_prefix + KT - 1) / KT + 1;
  if (want > tiles) want = tiles;
  if (want > 16) want = 16;
  return want < 1 ? 1 : want;
}

size_t attention_scratch_floats(const Dims& d, int batch, int splits) {
  return splits > 1 ? (size_t)batch * d.Hq * splits * QROWS * (d.dh + 2) : 0;
}

cudaError_t launch_attention_mma(const Request* rq, int* status, const float* qkv, const float2* rope, int layer,
                                 __nv_bfloat16* out_tiled, int rows_pad, int num_splits, float* scratch, const Dims& d,
                                 int batch, unsigned wait_limit, cudaStream_t st) {
  AttnArgs a{};
  a.rq = rq, a.status = status, a.qkv = qkv, a.rope = rope, a.layer = layer, a.out = out_tiled, a.rows_pad = rows_pad;
  a.num_splits = num_splits, a.d = d, a.wait_limit = wait_limit;
  a.part_o = scratch;
  a.part_ml = scratch ? scratch + (size_t)batch * d.Hq * num_splits * QROWS * d.dh : nullptr;
  const int G = d.Hq / d.Hkv;
  const bool two = (G % 2 == 0) && (batch * d.Hq * num_splits >= 2 * 148);
  // (one head per CTA with 32-key tiles, two CTAs per SM, was measured no faster than two heads per CTA)
  if (d.dh == 256) return two ? launch_attn<256, 2, 64>(a, batch, st) : launch_attn<256, 1, 64>(a, batch, st);
  if (d.dh == 128) return two ? launch_attn<128, 2, 64>(a, batch, st) : launch_attn<128, 1, 64>(a, batch, st);
  return two ? launch_attn<64, 2, 64>(a, batch, st) : launch_attn<64, 1, 64>(a, batch, st);
}

}  // namespace phyai

// =============================================================================================
// Stand-alone operator entry point
// =============================================================================================
namespace phyai {
namespace {

thread_local char g_op_err[256] = "";

// Shared body of the operator entry points: fills the request block at the head of `scratch`,
// then launches the attention (and merge) kernels with the split-KV partials placed after it.
phyai_status_t attention_op(const phyai_attention_desc_t* desc, uint32_t batch, const float* qkv, const void* prefix_kv,
                            uint64_t kv_tokens, const int32_t* cu, const float* rope, uint16_t* out, int32_t* status_word,
                            void* scratch, size_t scratch_bytes, cudaStream_t st) {
  auto bad = [](const char* m) {
    snprintf(g_op_err, sizeof(g_op_err), "%s", m);
    return PHYAI_ERR_INVALID_ARG;
  };
  if (!desc || desc->struct_size != sizeof(phyai_attention_desc_t)) return bad("desc is NULL or has a wrong struct_size");
  if (!qkv || !cu || !out || !status_word || !batch) return bad("qkv / cu_prefix_lens / out / status_word is NULL or batch is 0");
  if (kv_tokens && !prefix_kv) return bad("prefix_kv is NULL with kv_tokens > 0");
  if ((reinterpret_cast<uintptr_t>(prefix_kv) & 15u) || (reinterpret_cast<uintptr_t>(out) & 3u))
    return bad("prefix_kv must be 16-byte aligned and out 4-byte aligned");
  if (!desc->n_q_heads || !desc->n_kv_heads || desc->n_q_heads % desc->n_kv_heads || desc->layer >= desc->n_layers)
    return bad("head counts or layer index out of range");
  if (kv_tokens > (uint64_t)INT32_MAX || batch > 65535u) return bad("kv_tokens exceeds the int32 range or batch exceeds 65535");
  if (!desc->suffix_len) return bad("suffix_len is 0");
  Dims d{};
  d.L = (int)desc->n_layers, d.Hq = (int)desc->n_q_heads, d.Hkv = (int)desc->n_kv_heads, d.dh = (int)desc->head_dim;
  d.S = (int)desc->suffix_len, d.H = d.S, d.Nq = d.Hq * d.dh, d.Nqkv = (d.Hq + 2 * d.Hkv) * d.dh;
  d.block_causal = desc->state_token_block_causal ? 1 : 0, d.ns = d.block_causal;
  if (!attention_mma_supported(d)) {
    snprintf(g_op_err, sizeof(g_op_err), "head_dim must be 64, 128 or 256 and suffix_len <= 64");
    return PHYAI_ERR_UNSUPPORTED;
  }
  int splits = (int)desc->num_splits;
  if (splits == 0) splits = attention_pick_splits(d, (int)batch, (int)(kv_tokens < 4096 ? kv_tokens : 4096));
  if (splits < 1 || splits > 16) return bad("num_splits must be 0 (choose) or 1..16");
  const size_t need = 256 + attention_scratch_floats(d, (int)batch, splits) * sizeof(float);
  if (need > scratch_bytes) {
    snprintf(g_op_err, sizeof(g_op_err), "needs %zu bytes of scratch, only %zu available", need, scratch_bytes);
    return PHYAI_ERR_INVALID_ARG;
  }
  Request r{};
  r.prefix_kv = prefix_kv, r.kv_tokens = kv_tokens, r.cu_lens = cu, r.batch = (int)batch;
  Request* rq = reinterpret_cast<Request*>(scratch);
  launch_set_request(rq, r, nullptr, st);
  // cu_prefix_lens is checked on the device like in the denoise calls: a violation raises the caller's status word
  // (INVALID_ARG) and turns the attention kernels into no-ops
  launch_validate(rq, status_word, (int)kv_tokens, nullptr, st);
  float* partials = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(scratch) + 256);
  cudaError_t e = launch_attention_mma(rq, status_word, qkv, reinterpret_cast<const float2*>(rope), (int)desc->layer,
                                       reinterpret_cast<__nv_bfloat16*>(out), 0, splits, splits > 1 ? partials : nullptr,
                                       d, (int)batch, 1u << 22, st);
  if (e != cudaSuccess) {
    snprintf(g_op_err, sizeof(g_op_err), "attention launch failed: %s", cudaGetErrorString(e));
    return PHYAI_ERR_CUDA;
  }
  return PHYAI_OK;
}

}  // namespace
}  // namespace phyai

extern "C" {

const char* phyai_op_last_error(void) { return phyai::g_op_err; }

size_t phyai_suffix_attention_scratch_bytes(const phyai_attention_desc_t* desc, uint32_t batch) {
  if (!desc || !batch) return 0;
  phyai::Dims d{};
  d.Hq = (int)desc->n_q_heads, d.Hkv = (int)desc->n_kv_heads, d.dh = (int)desc->head_dim, d.S = (int)desc->suffix_len;
  const int splits = desc->num_splits ? (int)desc->num_splits : 16;
  return 256 + phyai::attention_scratch_floats(d, (int)batch, splits) * sizeof(float);
}

phyai_status_t phyai_suffix_attention(const phyai_attention_desc_t* desc, uint32_t batch, const float* qkv,
                                      const void* prefix_kv, uint64_t kv_tokens, const int32_t* cu_prefix_lens,
                                      const float* rope_cos_sin, uint16_t* out, int32_t* status_word, void* stream) {
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const size_t bytes = phyai_suffix_attention_scratch_bytes(desc, batch);
  if (!bytes) {
    snprintf(phyai::g_op_err, sizeof(phyai::g_op_err), "desc is NULL or batch is 0");
    return PHYAI_ERR_INVALID_ARG;
  }
  void* scratch = nullptr;
  cudaError_t e = cudaMallocAsync(&scratch, bytes, st);
  if (e != cudaSuccess) {
    snprintf(phyai::g_op_err, sizeof(phyai::g_op_err), "cudaMallocAsync(%zu) failed: %s", bytes, cudaGetErrorString(e));
    return PHYAI_ERR_OOM;
  }
  phyai_status_t s = phyai::attention_op(desc, batch, qkv, prefix_kv, kv_tokens, cu_prefix_lens, rope_cos_sin, out,
                                         status_word, scratch, bytes, st);
  cudaFreeAsync(scratch, st);  // stream-ordered: released after the kernels above have run
  return s;
}

}  // extern "C"

// =============================================================================================
// Attention operator that allocates nothing
// =============================================================================================
// Scratch for the request block and the split-KV partials lives in this fixed array instead of
// coming from an allocator.  Every GPU that loads the library holds it until the process exits.
#define PHYAI_STATIC_SCRATCH_BYTES (16u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[PHYAI_STATIC_SCRATCH_BYTES];

namespace phyai {
namespace {

std::mutex g_static_mu;
void* g_static_ptr[64] = {};  // per device: device address of g_static_scratch

// In host code `g_static_scratch` is only a stand-in for the symbol; the address a kernel can use
// has to be looked up once per device, with that device current.
phyai_status_t static_scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= 64) {
    snprintf(g_op_err, sizeof(g_op_err), "cudaGetDevice failed or device index %d is outside 0..63", dev);
    return PHYAI_ERR_CUDA;
  }
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) {
      snprintf(g_op_err, sizeof(g_op_err), "cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
      return PHYAI_ERR_CUDA;
    }
    g_static_ptr[dev] = p;
  }
  *out = g_static_ptr[dev];
  return PHYAI_OK;
}

}  // namespace
}  // namespace phyai

extern "C" {

size_t phyai_suffix_attention_static_capacity(void) { return PHYAI_STATIC_SCRATCH_BYTES; }

phyai_status_t phyai_suffix_attention_static(const phyai_attention_desc_t* desc, uint32_t batch, const float* qkv,
                                             const void* prefix_kv, uint64_t kv_tokens, const int32_t* cu_prefix_lens,
                                             const float* rope_cos_sin, uint16_t* out, int32_t* status_word,
                                             void* stream) {
  const size_t need = phyai_suffix_attention_scratch_bytes(desc, batch);
  if (!need) {
    snprintf(phyai::g_op_err, sizeof(phyai::g_op_err), "desc is NULL or batch is 0");
    return PHYAI_ERR_INVALID_ARG;
  }
  if (desc->num_splits != 0 && need > (size_t)PHYAI_STATIC_SCRATCH_BYTES) {
    snprintf(phyai::g_op_err, sizeof(phyai::g_op_err),
             "this shape needs %zu bytes of scratch but the built-in scratch holds %u: lower batch or num_splits, or "
             "use phyai_suffix_attention",
             need, PHYAI_STATIC_SCRATCH_BYTES);
    return PHYAI_ERR_INVALID_ARG;
  }
  void* scratch = nullptr;
  phyai_status_t s = phyai::static_scratch_address(&scratch);
  if (s != PHYAI_OK) return s;
  // attention_op re-derives the exact requirement (after choosing num_splits) and refuses sizes
  // beyond the capacity passed here.  Nothing in the scratch has to start at zero: the request
  // block is rewritten by every call and every partial that is read was written by the same call.
  return phyai::attention_op(desc, batch, qkv, prefix_kv, kv_tokens, cu_prefix_lens, rope_cos_sin, out, status_word,
                             scratch, PHYAI_STATIC_SCRATCH_BYTES, reinterpret_cast<cudaStream_t>(stream));
}

}  // extern "C"
