// Parameters and per-CTA plans of the persistent loop kernel (small batches: batch * suffix_len <= 64).
#pragma once

#include "kernels.h"

namespace phyai {

enum : int {
  MP_NORM1 = 0, MP_QKV, MP_ATTN, MP_MERGE, MP_O, MP_NORM2, MP_GATEUP, MP_DOWN,  // per layer
  MP_EMBED, MP_EMBED_GEMM, MP_FINAL,                                             // per step
  MP_COUNT
};

struct MegaGemmRole {
  int tile;       // 128-row tile of the packed weight matrix
  int kc_begin;   // first 64-wide k-chunk
  int kc_count;   // number of k-chunks (0 = this CTA has no role in the phase); <= 16
  int split;      // index of this k-range among the splits of the tile (selects the partial-sum slab)
};

struct MegaCtaPlan {
  MegaGemmRole qkv, o, gateup, down, embed_gemm;
  int norm_begin, norm_end;      // rows of the residual stream normalised by this CTA
  int attn_begin, attn_end;      // attention roles: id = (b * head_groups + hgrp) * splits + split
  int merge_begin, merge_end;    // merge roles: id = (b * Hq + head) * S + row
  int embed_begin, embed_end;    // action rows embedded by this CTA
  int final_begin, final_end;    // action rows whose velocity / Euler update this CTA computes
};

struct MegaParams {
  Dims d;
  int batch, M, n_steps, ada, sites, attn_splits, hpc;
  float dt;
  unsigned wait_limit;
  const Request* rq;
  int* status;
  unsigned* counters;            // [MP_COUNT], zeroed before every launch
  const MegaCtaPlan* plans;      // [gridDim.x]
  int n_cta[MP_COUNT];           // CTAs that signal each phase
  // packed bf16 weights, per-layer stride in bytes
  const __nv_bfloat16 *w_qkv, *w_o, *w_gu, *w_d, *w_embed;
  size_t stride_qkv, stride_o, stride_gu, stride_d;
  // per-output-channel scales (null = 1), per-layer stride in floats
  const float *s_qkv, *s_o, *s_g, *s_u, *s_d;
  // small fp32 tensors
  const float *Wc, *bcfold, *b2, *state_tok, *Wout, *bout;
  const float* gains;            // plain: [sites][D]
  const float* mod;              // ada:   [n_steps][sites][3D] (1+scale | shift | gate)
  const float* tb;               // pi0:   [n_steps][D]
  const float2* rope;
  // activations (tiled bf16 with rows_pad = 64 so that consecutive k-chunks are contiguous)
  float *h, *qkv;
  __nv_bfloat16 *xn64, *attn64, *m64, *u64;
  __nv_bfloat16 *qr, *kr, *vr;   // rotated (q also scaled) bf16 q [b][Hq][S][dh], k / v [b][Hkv][S][dh]
  float* attn_scratch;
  float* slab;                   // [max(o_splits, d_splits)][64][D] split-K partial sums of O / down
  int o_splits, d_splits;
  // optional trace: [gridDim.x][MP_COUNT][4] globaltimer stamps (ns) for the traced (step, layer):
  // worker inputs ready, worker role done, MMA issuer first activations, MMA issuer last MMA; null = off
  unsigned long long* trace;
  int trace_step, trace_layer;
};

// Host side ----------------------------------------------------------------------------------------
// True when the persistent kernel covers this shape (else the per-operator kernels are used).
bool mega_supported(const Dims& d, int batch);
int mega_attention_splits(const Dims& d, int batch, int max_prefix, int ncta);
// Fills plans[ncta] and n_cta[MP_COUNT]; returns false if the shape cannot be planned.
bool mega_plan(const Dims& d, int batch, int ada, int attn_splits, int ncta, MegaCtaPlan* plans, int* n_cta);
cudaError_t mega_setup(int head_dim);
cudaError_t launch_mega(const MegaParams& p, int ncta, cudaStream_t st);
size_t mega_scratch_floats(const Dims& d, int batch, int splits);

}  // namespace phyai
