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
  const float2* rope;    // [pos][dh/2] (cos, sin) or null
  int layer;
  __nv_bfloat16* out;    // tiled bf16 [Nq/64][rows_pad][64], or row-major [rows][Nq] when rows_pad <= 0
  int rows_pad;
  int num_splits;
  float* part_o;         // [b][head][split][64][DH] unnormalised
  float* part_ml;        // [b][head][split][64][2]  (max in log2 units, sum)
  Dims d;
  unsigned wait_limit;
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

// DH: head_dim; HPC: query heads per CTA (4 warps each).
template <int DH, int HPC>
__global__ void __launch_bounds__(HPC * 128, 1) k_attn_mma(const AttnArgs a) {
  constexpr int ROWB = DH * 2;                // bytes per row
  constexpr int CH = DH / 8;                  // 16-byte chunks per row
  constexpr int NTHREADS = HPC * 128;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  const uint32_t Qs = smem_u32(smem_raw);                         // [HPC*64] rows
  const uint32_t Ks = Qs + (uint32_t)HPC * QROWS * ROWB;          // [2][KT] rows
  const uint32_t Vs = Ks + 2u * KT * ROWB;                        // [2][KT] rows

  const Dims& d = a.d;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x, hgrp = blockIdx.y, b = blockIdx.z;
  const int head0 = hgrp * HPC;
  const int hk = head0 / (d.Hq / d.Hkv);
  const int S = d.S;
  if (status_set(a.status)) return;   // no block-wide waits depend on other blocks: a plain early exit is safe

  const Request r = *a.rq;
  const int p0 = r.cu_lens[b], P = r.cu_lens[b + 1] - p0;
  const int Tp = (P + KT - 1) / KT;          // prefix tiles; tile index Tp is the suffix tile
  const int T = Tp + 1;
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
    const int rows = min(KT, P - t * KT);
    const uint32_t kb = Ks + (uint32_t)buf * KT * ROWB, vb = Vs + (uint32_t)buf * KT * ROWB;
    for (int idx = tid; idx < KT * CH; idx += NTHREADS) {
      const int row = idx / CH, c = idx % CH;
      const bool ok = row < rows;
      const size_t g = (size_t)(t * KT + (ok ? row : 0)) * kv_stride + (size_t)c * 16;
      const uint32_t o = swz(row, c, ROWB);
      cp_async16(kb + o, Kg + g, ok ? 16u : 0u);
      cp_async16(vb + o, Vg + g, ok ? 16u : 0u);
    }
  };
  if (t_begin < t_end && t_begin < Tp) load_tile(t_begin, 0);
  cp_async_commit();

  // ---- Q: rotate, scale by dh^-1/2, round to bf16, into shared memory (4 column pairs per thread)
  const float qscale = rsqrtf((float)DH);
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

  for (int t = t_begin; t < t_end; ++t) {
    const int buf = (t - t_begin) & 1;
    const uint32_t Kb = Ks + (uint32_t)buf * KT * ROWB, Vb = Vs + (uint32_t)buf * KT * ROWB;
    int valid;  // keys of this tile that exist
    if (t + 1 < t_end && t + 1 < Tp) load_tile(t + 1, buf ^ 1);   // the other buffer was released by the
    cp_async_commit();                                            // barrier that ended the previous iteration
    if (t < Tp) {
      valid = min(KT, P - t * KT);
    } else {
      // -- suffix tile: rotate this request's own keys, round K and V to bf16
      valid = S;
      for (int idx = tid; idx < KT * (half / 4); idx += NTHREADS) {
        const int js = idx / (half / 4), j = (idx % (half / 4)) * 4;
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
        const uint32_t olo = swz(js, j >> 3, ROWB) + (j & 7) * 2, ohi = swz(js, (j + half) >> 3, ROWB) + (j & 7) * 2;
        asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(Kb + olo), "r"(pack_bf16(klo.x, klo.y)), "r"(pack_bf16(klo.z, klo.w)) : "memory");
        asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(Kb + ohi), "r"(pack_bf16(khi.x, khi.y)), "r"(pack_bf16(khi.z, khi.w)) : "memory");
        asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(Vb + olo), "r"(pack_bf16(vlo.x, vlo.y)), "r"(pack_bf16(vlo.z, vlo.w)) : "memory");
        asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(Vb + ohi), "r"(pack_bf16(vhi.x, vhi.y)), "r"(pack_bf16(vhi.z, vhi.w)) : "memory");
      }
    }
    cp_async_wait<1>();   // everything but the prefetch just issued has landed
    __syncthreads();      // tile t (copied or built above) and Q visible to all warps
    {
      // ---------------- S = Q K^T (16 rows x 64 keys per warp) ---------------------------------
      float s[KT / 8][4];
#pragma unroll
      for (int n = 0; n < KT / 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
      const uint32_t k_row = Kb + (uint32_t)((lane & 7) + (lane >> 4) * 8) * ROWB;
      const int k_c0 = (lane >> 3) & 1;
#pragma unroll 4
      for (int kk = 0; kk < DH / 16; ++kk) {
        uint32_t af[4];
        ldsm_x4(q_row + (uint32_t)(((kk * 2 + q_c0) ^ sw) << 4), af[0], af[1], af[2], af[3]);
        const uint32_t kofs = (uint32_t)(((kk * 2 + k_c0) ^ sw) << 4);
#pragma unroll
        for (int np = 0; np < KT / 16; ++np) {
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
      for (int n = 0; n < KT / 8; ++n) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int key = n * 8 + qd * 2 + (e & 1);
          const int row = (e < 2) ? row0 : row1;
          bool vis = key < valid;
          if (causal && row == 0 && key != 0) vis = false;  // state token sees only itself
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
      uint32_t pf[KT / 16][4];
#pragma unroll
      for (int n = 0; n < KT / 8; ++n) {
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
      for (int kj = 0; kj < KT / 16; ++kj) {
#pragma unroll
        for (int np = 0; np < DH / 16; ++np) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(v_row + (uint32_t)(kj * 16 * ROWB) + (uint32_t)(((np * 2 + v_c0) ^ sw) << 4), b0, b1, b2, b3);
          mma_bf16(o[2 * np], pf[kj], b0, b1);
          mma_bf16(o[2 * np + 1], pf[kj], b2, b3);
        }
      }
    }
    __syncthreads();  // everyone is done with `buf` before it is refilled
  }
  cp_async_wait<0>();

  // ---- finish: quad-reduce the row sums, write output or partial ----------------------------------------
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const int head = head0 + hl;
  if (a.num_splits == 1) {
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

// Combine the per-split partials: out = sum_s 2^(m_s - m) O_s / sum_s 2^(m_s - m) l_s.
template <int DH>
__global__ void k_attn_merge(const int* status, const float* part_o, const float* part_ml, __nv_bfloat16* out,
                             int rows_pad, int num_splits, int S, int Hq) {
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

template <int DH, int HPC>
constexpr size_t attn_smem() {
  return (size_t)(HPC * QROWS + 4 * KT) * DH * 2;
}

template <int DH, int HPC>
cudaError_t launch_attn(const AttnArgs& a, int batch, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(k_attn_mma<DH, HPC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)attn_smem<DH, HPC>());
    if (e != cudaSuccess) return e;
    configured = true;
  }
  dim3 grid(a.num_splits, a.d.Hq / HPC, batch);
  k_attn_mma<DH, HPC><<<grid, HPC * 128, attn_smem<DH, HPC>(), st>>>(a);
  if (a.num_splits > 1) {
    dim3 g2(a.d.S, a.d.Hq, batch);
    k_attn_merge<DH><<<g2, 128, 0, st>>>(a.status, a.part_o, a.part_ml, a.out, a.rows_pad, a.num_splits, a.d.S, a.d.Hq);
  }
  return cudaGetLastError();
}

}  // namespace

bool attention_mma_supported(const Dims& d) {
  return (d.dh == 64 || d.dh == 128 || d.dh == 256) && d.S <= QROWS;
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
  AttnArgs a;
  a.rq = rq, a.status = status, a.qkv = qkv, a.rope = rope, a.layer = layer, a.out = out_tiled, a.rows_pad = rows_pad;
  a.num_splits = num_splits, a.d = d, a.wait_limit = wait_limit;
  a.part_o = scratch;
  a.part_ml = scratch ? scratch + (size_t)batch * d.Hq * num_splits * QROWS * d.dh : nullptr;
  const int G = d.Hq / d.Hkv;
  const bool two = (G % 2 == 0) && (batch * d.Hq * num_splits >= 2 * 148);
  if (d.dh == 256) return two ? launch_attn<256, 2>(a, batch, st) : launch_attn<256, 1>(a, batch, st);
  if (d.dh == 128) return two ? launch_attn<128, 2>(a, batch, st) : launch_attn<128, 1>(a, batch, st);
  return two ? launch_attn<64, 2>(a, batch, st) : launch_attn<64, 1>(a, batch, st);
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
  if (kv_tokens > (uint64_t)INT32_MAX || batch > (1u << 16)) return bad("kv_tokens or batch too large");
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
