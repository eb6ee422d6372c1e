// Device-side body of the tensor-core suffix attention (one CTA-sized role), shared by the
// stand-alone kernel and the persistent loop kernel.
#pragma once

#include "kernels.h"
#include "ptx.cuh"
#include "tc.cuh"

namespace phyai {
namespace {

constexpr int KT = 64;      // keys per tile
constexpr int QROWS = 64;   // query rows per head (suffix length <= 64)
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Output element index: tiled bf16 when rows_pad > 0, else row-major with leading dimension ld.
__device__ __forceinline__ size_t out_index(int row, int col, int rows_pad, int ld) {
  return rows_pad > 0 ? tiled_index(row, col, rows_pad) : (size_t)row * ld + col;
}

struct AttnArgs {
  const Request* rq;
  int* status;
  const float* qkv;      // [rows][Nqkv] fp32 (q | k | v), un-rotated
  const __nv_bfloat16 *qr, *kr, *vr;  // or: rotated, scaled bf16 q [b][Hq][S][dh], k / v [b][Hkv][S][dh] (null = use qkv)
  const float2* rope;    // [pos][dh/2] (cos, sin) or null
  int layer;
  __nv_bfloat16* out;    // tiled bf16 [Nq/64][rows_pad][64], or row-major [rows][Nq] when rows_pad <= 0
  int rows_pad;
  int num_splits;
  float* part_o;         // [b][head][split][64][DH] unnormalised
  float* part_ml;        // [b][head][split][64][2]  (max in log2 units, sum)
  Dims d;
  unsigned wait_limit;
  const int* order;      // optional: request index of each grid row (batch entries)
  // fused output projection (cluster variant): CTA r of head h's cluster multiplies the merged head output by the
  // packed weight blocks (out-channel tile r, k-chunks of head h) and stores slab h of the split-K residual sum
  const __nv_bfloat16* wo;   // packed [D/128][Nq/64] blocks of 128 x 64
  const float* o_scale;      // per out channel, or null
  const float* o_gate;       // per out channel, or null
  float* slab;               // [Hq][rows][D]
  size_t slab_stride;        // rows * D
  int D;
  int trace_all;             // every CTA stamps, into slot (linear CTA index) of `trace`
  unsigned long long* trace; // cluster kernel: 16-entry slot or null: start, set-up done, Q acquired, tiles done, partials
                             // received, output written, cluster released
};
// shared-memory barriers and tensor-memory base of the fused output projection
struct OprojCtx {
  uint32_t x_bar, w_bar, mma_bar, tmem;
};

// Shared-memory tiles are rows of DH bf16 with no padding; the 16-byte chunk c of row r sits at
// chunk position c ^ (r & 7), which makes every ldmatrix (8 rows x 16 bytes) bank-conflict free.
__device__ __forceinline__ uint32_t swz(int row, int chunk, int rowb) {
  return (uint32_t)row * rowb + (uint32_t)((chunk ^ (row & 7)) << 4);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <int BAR, int NT>
__device__ __forceinline__ void group_sync() {
  asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(NT) : "memory");
}

// One attention role: the suffix rows of HPC query heads (head group `hgrp`) of request `b` against
// key tiles [T*split/num_splits, T*(split+1)/num_splits).  Executed by HPC*128 threads (`tid` is the
// thread's index within that group) that synchronise on named barrier BAR.  DH: head_dim; NBUF: K/V
// buffers (2 = prefetch the next tile during compute); KTT: keys per tile.  Shared memory at
// `smem_base` (128-byte aligned): (HPC*64 + 2*NBUF*KTT) rows of DH bf16.  When a.qr is set, q / k / v of
// the suffix are read as bf16, already rotated and scaled (written by the QKV epilogue of the
// persistent kernel); otherwise they are taken from the fp32 QKV output and rotated here.
// CLUSTER (HPC = 1): the num_splits = 8 key ranges of a head are the 8 CTAs of a thread-block cluster; each sends
// the rows of its partial (O, max, sum) into the shared memory of the CTA that owns them (bulk copies over
// distributed shared memory, counted on the owner's mbarrier) and every CTA merges its own 8 of the 64 rows: no
// partials in global memory, no merge kernel.  Needs 8 * 8 * (DH + 4) * 4 + 512 bytes of shared memory beyond the Q / K / V buffers.
template <int DH, int HPC, int NBUF, int BAR, int KTT, bool CLUSTER = false, bool OPROJ = false>
__device__ __forceinline__ void attn_role(const AttnArgs& a, int split, int hgrp, int b, uint32_t smem_base, int tid,
                                          uint32_t mrg_bar = 0, volatile int* abort_flag = nullptr,
                                          OprojCtx oc = OprojCtx{}) {
  constexpr int ROWB = DH * 2;                // bytes per row
  constexpr int CH = DH / 8;                  // 16-byte chunks per row
  constexpr int NTHREADS = HPC * 128;
  const uint32_t Qs = smem_base;                                  // [HPC*64] rows
  const uint32_t Ks = Qs + (uint32_t)HPC * QROWS * ROWB;          // [NBUF][KTT] rows
  const uint32_t Vs = Ks + (uint32_t)NBUF * KTT * ROWB;            // [NBUF][KTT] rows

  const Dims& d = a.d;
  const int warp = tid >> 5, lane = tid & 31;
  const int head0 = hgrp * HPC;
  const int hk = head0 / (d.Hq / d.Hkv);
  const int S = d.S;

  const Request r = *a.rq;
  const int p0 = r.cu_lens[b], P = r.cu_lens[b + 1] - p0;
  const int Tp = (P + KTT - 1) / KTT;          // prefix tiles, followed by the suffix tiles
  const int T = Tp + (S + KTT - 1) / KTT;
  const int t_begin = (int)(((long long)T * split) / a.num_splits);
  const int t_end = (int)(((long long)T * (split + 1)) / a.num_splits);

  const uint8_t* Kg = reinterpret_cast<const uint8_t*>(r.prefix_kv) +
                      (((size_t)(a.layer * 2 + 0) * r.kv_tokens + p0) * d.Hkv + hk) * ROWB;
  const uint8_t* Vg = reinterpret_cast<const uint8_t*>(r.prefix_kv) +
                      (((size_t)(a.layer * 2 + 1) * r.kv_tokens + p0) * d.Hkv + hk) * ROWB;
  const size_t kv_stride = (size_t)d.Hkv * ROWB;  // bytes between consecutive tokens
  constexpr int half = DH / 2;

  // K/V tile t -> buffer buf with 16-byte asynchronous copies; rows past the prefix are zero-filled
  auto load_tile = [&](int t, int buf) {
    const int rows = min(KTT, P - t * KTT);
    const uint32_t kb = Ks + (uint32_t)buf * KTT * ROWB, vb = Vs + (uint32_t)buf * KTT * ROWB;
    for (int idx = tid; idx < KTT * CH; idx += NTHREADS) {
      const int row = idx / CH, c = idx % CH;
      const bool ok = row < rows;
      const size_t g = (size_t)(t * KTT + (ok ? row : 0)) * kv_stride + (size_t)c * 16;
      const uint32_t o = swz(row, c, ROWB);
      cp_async16(kb + o, Kg + g, ok ? 16u : 0u);
      cp_async16(vb + o, Vg + g, ok ? 16u : 0u);
    }
  };
  if (t_begin < t_end && t_begin < Tp) load_tile(t_begin, 0);
  cp_async_commit();
  bool early2 = false;   // second key tile requested before the dependency wait (cluster variant)
  if constexpr (CLUSTER && NBUF == 2) {
    if (t_begin + 1 < t_end && t_begin + 1 < Tp) load_tile(t_begin + 1, 1), early2 = true;
    cp_async_commit();
  }
  // ---- per-warp state -----------------------------------------------------------------------------
  const int hl = warp >> 2, rb = warp & 3;             // local head, 16-row block
  const int g = lane >> 2, qd = lane & 3;              // row within 8, column pair
  const int row0 = rb * 16 + g, row1 = row0 + 8;       // this thread's two query rows
  const int sw = lane & 7;                             // swizzle term of every ldmatrix row this lane addresses
  float o[DH / 8][4];
#pragma unroll
  for (int n = 0; n < DH / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  const uint32_t q_row = Qs + (uint32_t)(hl * QROWS + rb * 16 + (lane & 15)) * ROWB;
  const int q_c0 = lane >> 4;

  // Everything that needs the kernel before this one: the dependency wait, Q, the status word.
  auto acquire_q = [&]() -> bool {
  if constexpr (CLUSTER) {
    // Programmatic dependent launch: the request block and the prefix K/V were complete before this grid could
    // start, so the first key tile is already on its way; q / k / v of the suffix come from the kernel before.
    pdl_wait();
  }

  if (a.qr) {
    // ---- Q rows are ready-made bf16: straight asynchronous copies (rows past the suffix are zero-filled)
    for (int idx = tid; idx < HPC * QROWS * CH; idx += NTHREADS) {
      const int hl = idx / (QROWS * CH), rem = idx % (QROWS * CH);
      const int i = rem / CH, c = rem % CH;
      const bool ok = i < S;
      const uint8_t* src = reinterpret_cast<const uint8_t*>(a.qr) +
                           ((size_t)((b * d.Hq + head0 + hl) * S + (ok ? i : 0)) * CH + c) * 16;
      cp_async16(Qs + swz(hl * QROWS + i, c, ROWB), src, ok ? 16u : 0u);
    }
    cp_async_commit();
  }
  if constexpr (CLUSTER) {
    // The status word is read after the Q copies have been requested (their addresses do not depend on the request),
    // so that its round trip to the L2 overlaps theirs.
    if (status_set(a.status)) {   // same answer in every CTA of the cluster (all earlier kernels have completed)
      cp_async_wait<0>();
      return false;
    }
  }
  // ---- Q: rotate, scale by dh^-1/2, round to bf16, into shared memory (4 column pairs per thread)
  const float qscale = rsqrtf((float)DH);
  if (!a.qr)
#pragma unroll 4
  for (int idx = tid; idx < HPC * QROWS * (half / 4); idx += NTHREADS) {
    const int hl = idx / (QROWS * (half / 4)), rem = idx % (QROWS * (half / 4));
    const int i = rem / (half / 4), j = (rem % (half / 4)) * 4;
    float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
    if (i < S) {
      const float* q = a.qkv + (size_t)(b * S + i) * d.Nqkv + (size_t)(head0 + hl) * DH;
      lo = *reinterpret_cast<const float4*>(q + j);
      hi = *reinterpret_cast<const float4*>(q + j + half);
      if (a.rope) {
        const float4 cs0 = *reinterpret_cast<const float4*>(a.rope + (size_t)(P + i) * half + j);
        const float4 cs1 = *reinterpret_cast<const float4*>(a.rope + (size_t)(P + i) * half + j + 2);
        const float4 l2 = make_float4(lo.x * cs0.x - hi.x * cs0.y, lo.y * cs0.z - hi.y * cs0.w,
                                      lo.z * cs1.x - hi.z * cs1.y, lo.w * cs1.z - hi.w * cs1.w);
        hi = make_float4(hi.x * cs0.x + lo.x * cs0.y, hi.y * cs0.z + lo.y * cs0.w, hi.z * cs1.x + lo.z * cs1.y,
                         hi.w * cs1.z + lo.w * cs1.w);
        lo = l2;
      }
    }
    const int row = hl * QROWS + i;
    const uint2 plo = make_uint2(pack_bf16(lo.x * qscale, lo.y * qscale), pack_bf16(lo.z * qscale, lo.w * qscale));
    const uint2 phi = make_uint2(pack_bf16(hi.x * qscale, hi.y * qscale), pack_bf16(hi.z * qscale, hi.w * qscale));
    asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(Qs + swz(row, j >> 3, ROWB) + (j & 7) * 2), "r"(plo.x), "r"(plo.y) : "memory");
    asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(Qs + swz(row, (j + half) >> 3, ROWB) + (j & 7) * 2), "r"(phi.x), "r"(phi.y) : "memory");
  }

    return true;
  };
  // Cluster variant: the tile loop makes one extra pass, before the dependency wait, over whatever the buffers hold
  // (results discarded).  The kernel starts long before its dependency resolves, and the first pass through this
  // code was measured ~1 us slower than later ones.
  bool acquired = false;
  if constexpr (!CLUSTER) {
    acquire_q();
    acquired = true;
  }
#pragma unroll 1
  for (int t = CLUSTER ? t_begin - 1 : t_begin; t < t_end; ++t) {
    const bool warm = CLUSTER && t < t_begin;
    if (CLUSTER && t == t_begin) {
      if (!acquire_q()) return;
      acquired = true;
      if (tid == 0 && split == 0 && hgrp == 0 && b == 0) trace_stamp(a.trace, 2);
#pragma unroll
      for (int n = 0; n < DH / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
      m0 = m1 = -INFINITY, l0 = l1 = 0.f;
    }
    const int buf = NBUF == 2 ? ((t - t_begin) & 1) : 0;
    const uint32_t Kb = Ks + (uint32_t)buf * KTT * ROWB, Vb = Vs + (uint32_t)buf * KTT * ROWB;
    int valid;  // keys of this tile that exist
    if (NBUF == 2 && !warm) {
      if (t + 1 < t_end && t + 1 < Tp && !(early2 && t == t_begin)) load_tile(t + 1, buf ^ 1);   // the other buffer was released by the
      cp_async_commit();                                            // barrier that ended the previous iteration
    }
    if (warm) {
      valid = KTT;
    } else if (t < Tp) {
      valid = min(KTT, P - t * KTT);
    } else if (a.qr) {
      // -- suffix tile from the ready-made bf16 keys / values
      const int j0 = (t - Tp) * KTT;
      valid = min(KTT, S - j0);
      const uint8_t* ksrc = reinterpret_cast<const uint8_t*>(a.kr) + (size_t)((b * d.Hkv + hk) * S + j0) * ROWB;
      const uint8_t* vsrc = reinterpret_cast<const uint8_t*>(a.vr) + (size_t)((b * d.Hkv + hk) * S + j0) * ROWB;
      for (int idx = tid; idx < KTT * CH; idx += NTHREADS) {
        const int row = idx / CH, c = idx % CH;
        const bool ok = row < valid;
        const size_t g = (size_t)(ok ? row : 0) * ROWB + (size_t)c * 16;
        cp_async16(Kb + swz(row, c, ROWB), ksrc + g, ok ? 16u : 0u);
        cp_async16(Vb + swz(row, c, ROWB), vsrc + g, ok ? 16u : 0u);
      }
      cp_async_commit();
    } else {
      // -- suffix tile: rotate this request's own keys, round K and V to bf16
      const int j0 = (t - Tp) * KTT;
      valid = min(KTT, S - j0);
#pragma unroll 2
      for (int idx = tid; idx < KTT * (half / 4); idx += NTHREADS) {
        const int lr = idx / (half / 4), js = j0 + lr, j = (idx % (half / 4)) * 4;
        float4 klo = make_float4(0.f, 0.f, 0.f, 0.f), khi = klo, vlo = klo, vhi = klo;
        if (js < S) {
          const float* kr = a.qkv + (size_t)(b * S + js) * d.Nqkv + d.Nq + (size_t)hk * DH;
          const float* vr = kr + d.Hkv * DH;
          klo = *reinterpret_cast<const float4*>(kr + j), khi = *reinterpret_cast<const float4*>(kr + j + half);
          vlo = *reinterpret_cast<const float4*>(vr + j), vhi = *reinterpret_cast<const float4*>(vr + j + half);
          if (a.rope) {
            const float4 cs0 = *reinterpret_cast<const float4*>(a.rope + (size_t)(P + js) * half + j);
            const float4 cs1 = *reinterpret_cast<const float4*>(a.rope + (size_t)(P + js) * half + j + 2);
            const float4 l2 = make_float4(klo.x * cs0.x - khi.x * cs0.y, klo.y * cs0.z - khi.y * cs0.w,
                                          klo.z * cs1.x - khi.z * cs1.y, klo.w * cs1.z - khi.w * cs1.w);
            khi = make_float4(khi.x * cs0.x + klo.x * cs0.y, khi.y * cs0.z + klo.y * cs0.w,
                              khi.z * cs1.x + klo.z * cs1.y, khi.w * cs1.z + klo.w * cs1.w);
            klo = l2;
          }
        }
        const uint32_t olo = swz(lr, j >> 3, ROWB) + (j & 7) * 2, ohi = swz(lr, (j + half) >> 3, ROWB) + (j & 7) * 2;
        asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(Kb + olo), "r"(pack_bf16(klo.x, klo.y)), "r"(pack_bf16(klo.z, klo.w)) : "memory");
        asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(Kb + ohi), "r"(pack_bf16(khi.x, khi.y)), "r"(pack_bf16(khi.z, khi.w)) : "memory");
        asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(Vb + olo), "r"(pack_bf16(vlo.x, vlo.y)), "r"(pack_bf16(vlo.z, vlo.w)) : "memory");
        asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(Vb + ohi), "r"(pack_bf16(vhi.x, vhi.y)), "r"(pack_bf16(vhi.z, vhi.w)) : "memory");
      }
    }
    if (warm) {
      // (nothing to wait for: this pass only exercises the code)
    } else if (NBUF == 2 && !(a.qr && t >= Tp)) {
      cp_async_wait<1>();   // everything but the prefetch just issued has landed
    } else {
      cp_async_wait<0>();
    }
    group_sync<BAR, NTHREADS>();         // tile t (copied or built above) and Q visible to all warps
    {
      // ---------------- S = Q K^T (16 rows x KTT keys per warp) ---------------------------------
      float s[KTT / 8][4];
#pragma unroll
      for (int n = 0; n < KTT / 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
      const uint32_t k_row = Kb + (uint32_t)((lane & 7) + (lane >> 4) * 8) * ROWB;
      const int k_c0 = (lane >> 3) & 1;
#pragma unroll 4
      for (int kk = 0; kk < DH / 16; ++kk) {
        uint32_t af[4];
        ldsm_x4(q_row + (uint32_t)(((kk * 2 + q_c0) ^ sw) << 4), af[0], af[1], af[2], af[3]);
        const uint32_t kofs = (uint32_t)(((kk * 2 + k_c0) ^ sw) << 4);
#pragma unroll
        for (int np = 0; np < KTT / 16; ++np) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4(k_row + (uint32_t)(np * 16 * ROWB) + kofs, b0, b1, b2, b3);
          mma_bf16(s[2 * np], af, b0, b1);
          mma_bf16(s[2 * np + 1], af, b2, b3);
        }
      }
      // ---------------- mask + online softmax (log2 domain) ----------------------------------------
      const bool suffix_tile = t >= Tp;
      const bool causal = suffix_tile && d.block_causal && d.ns;
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int n = 0; n < KTT / 8; ++n) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int key = n * 8 + qd * 2 + (e & 1);
          const int row = (e < 2) ? row0 : row1;
          bool vis = key < valid;
          if (causal && row == 0 && (t - Tp) * KTT + key != 0) vis = false;  // state token sees only itself
          s[n][e] = vis ? s[n][e] * LOG2E : -INFINITY;
        }
        mx0 = fmaxf(mx0, fmaxf(s[n][0], s[n][1]));
        mx1 = fmaxf(mx1, fmaxf(s[n][2], s[n][3]));
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
      const float c0 = (mn0 == -INFINITY) ? 1.f : exp2f(m0 - mn0);
      const float c1 = (mn1 == -INFINITY) ? 1.f : exp2f(m1 - mn1);
      const float sub0 = (mn0 == -INFINITY) ? 0.f : mn0, sub1 = (mn1 == -INFINITY) ? 0.f : mn1;
      m0 = mn0, m1 = mn1;
      float rs0 = 0.f, rs1 = 0.f;
      uint32_t pf[KTT / 16][4];
#pragma unroll
      for (int n = 0; n < KTT / 8; ++n) {
        const float p0 = exp2f(s[n][0] - sub0), p1 = exp2f(s[n][1] - sub0);
        const float p2 = exp2f(s[n][2] - sub1), p3 = exp2f(s[n][3] - sub1);
        rs0 += p0 + p1, rs1 += p2 + p3;
        pf[n >> 1][(n & 1) * 2 + 0] = pack_bf16(p0, p1);
        pf[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
      }
      l0 = l0 * c0 + rs0, l1 = l1 * c1 + rs1;
#pragma unroll
      for (int n = 0; n < DH / 8; ++n) {
        o[n][0] *= c0, o[n][1] *= c0, o[n][2] *= c1, o[n][3] *= c1;
      }
      // ---------------- O += P V ----------------------------------------------------------------------
      const uint32_t v_row = Vb + (uint32_t)((lane & 7) + ((lane >> 3) & 1) * 8) * ROWB;
      const int v_c0 = lane >> 4;
#pragma unroll
      for (int kj = 0; kj < KTT / 16; ++kj) {
#pragma unroll
        for (int np = 0; np < DH / 16; ++np) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(v_row + (uint32_t)(kj * 16 * ROWB) + (uint32_t)(((np * 2 + v_c0) ^ sw) << 4), b0, b1, b2, b3);
          mma_bf16(o[2 * np], pf[kj], b0, b1);
          mma_bf16(o[2 * np + 1], pf[kj], b2, b3);
        }
      }
    }
    group_sync<BAR, NTHREADS>();  // everyone is done with `buf` before it is refilled
    if (NBUF == 1) {
      if (t + 1 < t_end && t + 1 < Tp) load_tile(t + 1, 0);
      cp_async_commit();
    }
  }
  cp_async_wait<0>();
  if (CLUSTER && tid == 0 && split == 0 && hgrp == 0 && b == 0) trace_stamp(a.trace, 3);
  if constexpr (CLUSTER) {
    if (!acquired) {   // no key tile for this CTA: it still takes part in the merge, with an empty partial
      if (!acquire_q()) return;
#pragma unroll
      for (int n = 0; n < DH / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
      m0 = m1 = -INFINITY, l0 = l1 = 0.f;
    }
  }

  // ---- finish: quad-reduce the row sums, write output or partial ----------------------------------------
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const int head = head0 + hl;
  if constexpr (CLUSTER) {
    // Push merge: CTA `rank` of the cluster owns rows [8 * rank, 8 * rank + 8).  Every CTA sends the owners their
    // rows of its partial (and their max / sum), into a receive area beyond the Q / K / V buffers, which the owner
    // may still be using; each CTA then merges its 8 rows from its own shared memory.
    constexpr int PP = DH + 4;                       // row pitch in floats
    constexpr uint32_t OWN_BYTES = 8u * PP * 4u;     // one owner's 8 rows of a partial
    const uint32_t recv = smem_base + (uint32_t)(HPC * QROWS + 2 * NBUF * KTT) * ROWB;   // [8 sources][8 rows][PP]
    const uint32_t recv_ml = recv + 8u * OWN_BYTES;                                       // [8 sources][8 rows][2]
    // The partial is first written to this CTA's own shared memory (over the K / V buffers, which every thread has
    // finished with: the tile loop ends with a barrier), grouped by owner, then sent with one bulk copy per owner
    // (distributed shared memory, completion counted on the owner's mbarrier): remote stores from the threads
    // themselves measured ~3 us for the 64 KB.
    // (with the fused projection the staging area starts at the Q buffer instead, which is dead as well: the V
    // buffers then take the projection's weight blocks and the tail of the K buffers its activation tile)
    const uint32_t stg = OPROJ ? Qs : Ks, stg_ml = stg + 8u * OWN_BYTES;
    constexpr uint32_t XK = 7u * 1024u;                                     // k-chunk pitch of the activation tile: 56 rows
    const uint32_t xt = smem_base + ((8u * OWN_BYTES + 512u + 1023u) & ~1023u);   // [4][56 rows][128 B], swizzled
    if constexpr (OPROJ) {
      static_assert(DH == 256 && KTT == 64 && HPC == 1 && NBUF == 2, "fused projection: head_dim 256 only");
      if (tid == 0) {
        // the four 128 x 64 weight blocks of (out-channel tile = my rank, k-chunks of my head): 64 KB, contiguous
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        const uint8_t* wsrc = reinterpret_cast<const uint8_t*>(a.wo) + ((size_t)split * (a.d.Nq / 64) + (size_t)head * 4) * 16384;
        mbar_expect_tx(oc.w_bar, 65536u);
#pragma unroll
        for (int c = 0; c < 4; ++c) bulk_g2s(Vs + (uint32_t)c * 16384u, wsrc + (size_t)c * 16384, 16384u, oc.w_bar);
      }
    }
#pragma unroll
    for (int n = 0; n < DH / 8; ++n) {
      const uint32_t col = (uint32_t)(n * 8 + qd * 2) * 4;
      asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(stg + (uint32_t)(row0 * PP) * 4 + col), "f"(o[n][0]), "f"(o[n][1]) : "memory");
      asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(stg + (uint32_t)(row1 * PP) * 4 + col), "f"(o[n][2]), "f"(o[n][3]) : "memory");
    }
    if (qd == 0) {
      asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(stg_ml + (uint32_t)row0 * 8), "f"(m0), "f"(l0) : "memory");
      asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(stg_ml + (uint32_t)row1 * 8), "f"(m1), "f"(l1) : "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the bulk-copy engine
    group_sync<BAR, NTHREADS>();
    if (tid < 16) {
      const uint32_t owner = (uint32_t)tid & 7u, ml = (uint32_t)tid >> 3;
      const uint32_t src = ml ? stg_ml + owner * 64u : stg + owner * OWN_BYTES;
      const uint32_t bytes = ml ? 64u : OWN_BYTES;
      const uint32_t dst_local = ml ? recv_ml + (uint32_t)split * 64u : recv + (uint32_t)split * OWN_BYTES;
      uint32_t dst, bar;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"(dst_local), "r"(owner));
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar) : "r"(mrg_bar), "r"(owner));
      asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                   "r"(src), "r"(bytes), "r"(bar)
                   : "memory");
    }
    {
      const WaitCtx wc{a.status, abort_flag, a.wait_limit};
      mbar_wait_drain(mrg_bar, 0u, wc);     // all eight partials of my rows have landed in `recv`
    }
    if (tid == 0 && split == 0 && hgrp == 0 && b == 0) trace_stamp(a.trace, 4);
    constexpr int CPT = DH / 16;                                  // columns per thread: 16 threads cover a row
    const int rl = tid >> 4, r = split * 8 + rl, c0 = (tid & 15) * CPT;
    if (r < S) {
      float ms[8], ls[8], mm = -INFINITY;
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(ms[s]), "=f"(ls[s]) : "r"(recv_ml + (uint32_t)(s * 8 + rl) * 8) : "memory");
        mm = fmaxf(mm, ms[s]);
      }
      float acc[CPT], ll = 0.f;
#pragma unroll
      for (int e = 0; e < CPT; ++e) acc[e] = 0.f;
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        if (ms[s] == -INFINITY) continue;
        const float w = exp2f(ms[s] - mm);
        ll = fmaf(w, ls[s], ll);
#pragma unroll
        for (int u = 0; u < CPT / 4; ++u) {
          float4 v;
          asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                       : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                       : "r"(recv + (uint32_t)((s * 8 + rl) * PP + c0 + 4 * u) * 4)
                       : "memory");
          acc[4 * u] = fmaf(w, v.x, acc[4 * u]), acc[4 * u + 1] = fmaf(w, v.y, acc[4 * u + 1]);
          acc[4 * u + 2] = fmaf(w, v.z, acc[4 * u + 2]), acc[4 * u + 3] = fmaf(w, v.w, acc[4 * u + 3]);
        }
      }
      const float inv = 1.0f / ll;
      if constexpr (OPROJ) {
        // my 16 columns of row r, as two 16-byte groups of k-chunk (tid & 15) / 4 of the projection's activation tile
        const uint32_t base = xt + (uint32_t)((tid & 15) >> 2) * XK + (uint32_t)r * 128u;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const uint32_t grp = (uint32_t)((tid & 3) * 2 + u) ^ (uint32_t)(r & 7);
          asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(base + grp * 16u),
                       "r"(pack_bf16(acc[8 * u] * inv, acc[8 * u + 1] * inv)), "r"(pack_bf16(acc[8 * u + 2] * inv, acc[8 * u + 3] * inv)),
                       "r"(pack_bf16(acc[8 * u + 4] * inv, acc[8 * u + 5] * inv)), "r"(pack_bf16(acc[8 * u + 6] * inv, acc[8 * u + 7] * inv))
                       : "memory");
        }
      } else {
#pragma unroll
      for (int u = 0; u < CPT / 4; ++u)     // 4 consecutive columns = 8 bytes, inside one 16-byte chunk of the tiled layout
        *reinterpret_cast<uint2*>(a.out + out_index(b * S + r, head * DH + c0 + 4 * u, a.rows_pad, d.Nq)) =
            make_uint2(pack_bf16(acc[4 * u] * inv, acc[4 * u + 1] * inv), pack_bf16(acc[4 * u + 2] * inv, acc[4 * u + 3] * inv));
      }
    }
    if constexpr (OPROJ) {
      const WaitCtx wc{a.status, abort_flag, a.wait_limit};
      // ---- all-gather of the merged rows: my rows go from my activation tile into the same place of every peer's
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      group_sync<BAR, NTHREADS>();
      const int nr = max(0, min(8, S - split * 8));            // rows I own
      if (tid < 32 && (tid & 7) != split && nr > 0) {
        const uint32_t peer = (uint32_t)tid & 7u, kc = (uint32_t)tid >> 3;
        const uint32_t loc = xt + kc * XK + (uint32_t)split * 1024u;
        uint32_t dst, bar;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"(loc), "r"(peer));
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar) : "r"(oc.x_bar), "r"(peer));
        asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                     "r"(loc), "r"((uint32_t)nr * 128u), "r"(bar)
                     : "memory");
      }
      // ---- D[128 out channels][64 tokens] = W[128][256] X^T: 16 MMAs issued by warp 0
      constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
      if (warp == 0) {
        const bool okx = mbar_wait_drain(oc.x_bar, 0u, wc) > 0;
        const bool okw = mbar_wait_drain(oc.w_bar, 0u, wc) > 0;
        tc_fence_after();
        if (__all_sync(0xffffffffu, okx && okw)) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint64_t da = make_desc(Vs + (uint32_t)c * 16384u), db = make_desc(xt + (uint32_t)c * XK);
#pragma unroll
            for (int k = 0; k < 4; ++k)
              if (elect_one()) umma_bf16(oc.tmem, da + 2 * k, db + 2 * k, IDESC, (c | k) ? 1u : 0u);
          }
        }
        if (elect_one()) umma_commit(oc.mma_bar);
        __syncwarp();
      }
      // ---- epilogue: accumulator -> slab `head`.  A warp holds 32 consecutive out channels of every token, so
      // its stores are whole 128-byte lines without a transpose.
      const int ch = warp * 32 + lane;                       // TMEM lane = out channel within the tile
      const int n = split * 128 + ch;
      const float sc = (a.o_scale ? a.o_scale[n] : 1.0f) * (a.o_gate ? a.o_gate[n] : 1.0f);
      const bool okm = mbar_wait_drain(oc.mma_bar, 0u, wc) > 0;
      tc_fence_after();
      if (okm) {
        float* dst = a.slab + (size_t)head * a.slab_stride + (size_t)(b * S) * a.D + n;
        for (int c0 = 0; c0 < S; c0 += 16) {
          float v[16];
          tmem_ld16(oc.tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (c0 + j < S) dst[(size_t)(c0 + j) * a.D] = v[j] * sc;
        }
      }
      tc_fence_before();
    }
    if (tid == 0 && split == 0 && hgrp == 0 && b == 0) trace_stamp(a.trace, 5);
    // every CTA has received everything by now, i.e. every outgoing copy has finished reading its source: only
    // then may a CTA leave and release its shared memory
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (tid == 0 && split == 0 && hgrp == 0 && b == 0) trace_stamp(a.trace, 6);
  } else if (a.num_splits == 1) {
    const float i0 = 1.0f / l0, i1 = 1.0f / l1;
#pragma unroll
    for (int n = 0; n < DH / 8; ++n) {
      const int col = head * DH + n * 8 + qd * 2;
      if (row0 < S)
        *reinterpret_cast<uint32_t*>(a.out + out_index(b * S + row0, col, a.rows_pad, d.Nq)) =
            pack_bf16(o[n][0] * i0, o[n][1] * i0);
      if (row1 < S)
        *reinterpret_cast<uint32_t*>(a.out + out_index(b * S + row1, col, a.rows_pad, d.Nq)) =
            pack_bf16(o[n][2] * i1, o[n][3] * i1);
    }
  } else {
    const size_t slab = ((size_t)(b * d.Hq + head) * a.num_splits + split) * QROWS;
    float* po = a.part_o + slab * DH;
    float* pm = a.part_ml + slab * 2;
#pragma unroll
    for (int n = 0; n < DH / 8; ++n) {
      const int col = n * 8 + qd * 2;
      if (row0 < S) *reinterpret_cast<float2*>(po + (size_t)row0 * DH + col) = make_float2(o[n][0], o[n][1]);
      if (row1 < S) *reinterpret_cast<float2*>(po + (size_t)row1 * DH + col) = make_float2(o[n][2], o[n][3]);
    }
    if (qd == 0) {
      if (row0 < S) pm[row0 * 2] = m0, pm[row0 * 2 + 1] = l0;
      if (row1 < S) pm[row1 * 2] = m1, pm[row1 * 2 + 1] = l1;
    }
  }
}

// Stand-alone kernel: grid (splits, head groups, requests).
template <int DH, int HPC, int KTT>
__global__ void __launch_bounds__(HPC * 128, 1) k_attn_mma(const AttnArgs a) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  pdl_enter();
  if (status_set(a.status)) return;   // no wait in this kernel depends on another block: a plain exit is safe
  attn_role<DH, HPC, 2, 0, KTT>(a, blockIdx.x, blockIdx.y, blockIdx.z, smem_u32(smem_raw), threadIdx.x);
}

// Cluster variant: grid (8, heads, requests), cluster (8, 1, 1); see attn_role.  OPROJ: the output projection of
// the head follows in the same kernel (tcgen05, accumulator in tensor memory) and leaves as slab `head` of the
// split-K residual sum, so the merged attention output never goes to global memory.
template <int DH, int KTT, bool OPROJ = false>
__global__ void __launch_bounds__(128, 1) k_attn_cluster(const AttnArgs a) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t mrg_bar;
  __shared__ __align__(8) uint64_t op_bar[3];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  pdl_launch_dependents();            // (the dependency wait and the status check are inside the role)
  const bool tracer = threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0;
  if (tracer) trace_stamp(a.trace, 0);
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&mrg_bar), 1);
    mbar_expect_tx(smem_u32(&mrg_bar), 8u * (8u * (DH + 4) * 4u + 64u));   // eight sources: 8 rows of O and of (max, sum)
    if (OPROJ) {
      for (int i = 0; i < 3; ++i) mbar_init(smem_u32(&op_bar[i]), 1);
      // merged rows of the seven peers: every row of the suffix but my own, four 128-byte pieces each
      const int mine = max(0, min(8, a.d.S - (int)blockIdx.x * 8));
      mbar_expect_tx(smem_u32(&op_bar[0]), (uint32_t)(a.d.S - mine) * 512u);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  OprojCtx oc{};
  if (OPROJ) {
    if (threadIdx.x < 32) {
      tmem_alloc(smem_u32(&tmem_slot), 64);
      tc_fence_before();
    }
  }
  // every CTA's barriers exist before any peer can send to them (this runs before the dependency wait)
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  if (tracer) trace_stamp(a.trace, 1);
  if (OPROJ) {
    __syncthreads();
    tc_fence_after();
    oc.x_bar = smem_u32(&op_bar[0]), oc.w_bar = smem_u32(&op_bar[1]), oc.mma_bar = smem_u32(&op_bar[2]);
    oc.tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  }
  // (the projection's operands need 1024-byte aligned tiles: the launch adds 1 KB of slack for this)
  const uint32_t smem_base = OPROJ ? ((smem_u32(smem_raw) + 1023u) & ~1023u) : smem_u32(smem_raw);
  attn_role<DH, 1, 2, 0, KTT, true, OPROJ>(a, blockIdx.x, blockIdx.y, blockIdx.z, smem_base, threadIdx.x,
                                           smem_u32(&mrg_bar), &abort_flag, oc);
  if (OPROJ) {
    __syncthreads();
    if (threadIdx.x < 32) {
      tc_fence_after();
      tmem_dealloc(oc.tmem, 64);
    }
  }
}

}  // namespace
}  // namespace phyai
