// Step boundary of the single-token-tile loop (at most 64 suffix tokens in the call, model width 1024): one cluster of
// 8 CTAs does what sits between the last layer of Euler step k - 1 and the first layer of step k (Sec. "action expert":
// final norm, velocity head, x <- x + dt v; then the suffix embedding of the updated actions).
//
//   stage 1  CTA c takes channels [128 c, 128 c + 128) of the residual stream of every token row: with the norm's
//            1 / rms factored out of the contraction, v[r][a] = rs[r] * sum_d (h[r][d] gain[d]) Wout[d][a]
//            + sum_d shift[d] Wout[d][a] + bout[a].  The CTA forms its slice of the first sum (tf32 mma.sync, the Wout
//            slice in registers as B fragments, fetched ahead of the dependency wait), its slice of sum_d h[r][d]^2 and
//            of the shift term.  Token row r belongs to CTA r mod 8: the partials of a CTA's rows travel to it as one
//            bulk copy per peer over distributed shared memory (a reduce-scatter by rows), are added in CTA order,
//            and the owner applies the Euler update to its rows.
//   stage 2  the owner embeds its (at most 8) rows over all 1024 channels (tf32 mma.sync, Wc in shared memory, fetched
//            ahead of the dependency wait): pi0 -- u = swish(x Wc + tb_k), the folded action / time MLP's first layer,
//            written as the bf16 tile of the second layer's projection; pi0.5 -- h = x Wa + ba and, for layer 0's
//            folded norm, bf16(h * gain) and the row's sum of squares.
//
// tf32 keeps 10 mantissa bits of each operand (more than the bf16 operands of every other projection of this path);
// sums are fp32.  The first call of a denoise (`first`) has no stage 1, the last (`last`) no stage 2.  The one wait on
// other CTAs' progress (the partials) is bounded; no CTA leaves before the closing cluster barrier.
#include "common.cuh"
#include "kernels.h"
#include "ptx.cuh"

namespace phyai {
namespace {

constexpr int SB_MAXA = 32;                 // action width
constexpr int SB_NC = 8;                    // CTAs of the cluster = 128-channel slices of the model width
constexpr int SB_D = SB_NC * 128;
constexpr int SB_THREADS = 512, SB_WARPS = 16;
constexpr int HS = 132;                     // row stride (floats) of the h slice: conflict-free A-fragment reads
constexpr int XS = 36;                      // row stride of the action rows
constexpr int WS = SB_D + 8;                // row stride of Wc in shared memory: conflict-free B-fragment reads
constexpr int PS = 33;                      // a partial's row: 32 velocities + the sum of squares
constexpr int PBLOCK = 300;                 // floats sent to one owner: its 8 rows + the shift-term row, 16-byte padded
constexpr uint32_t PBYTES = PBLOCK * 4;

__device__ __forceinline__ uint32_t sb_cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void sb_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t tf32_of(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}
// D(16x8) += A(16x8, row) B(8x8, col), tf32 operands, fp32 accumulation
__device__ __forceinline__ void mma_tf32(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__global__ void __launch_bounds__(SB_THREADS, 1) k_step_b1(int* status, const StepB1 p) {
  extern __shared__ __align__(16) float sb_smem[];
  __shared__ __align__(8) uint64_t bar_recv;
  __shared__ int abort_flag, recv_ok;
  constexpr int D = SB_D, NC = SB_NC;
  const int A = p.A;
  float* h_s = sb_smem;                         // [64][HS]   tf32(h * gain) of my 128 channels
  float* part = h_s + 64 * HS;                  // [8 owners][PBLOCK] my partial: rows local * 33 + col, shift row at 8 * 33
  float* recv = part + NC * PBLOCK;             // [8 sources][PBLOCK]
  float* xt = recv + NC * PBLOCK;               // [8 rows of mine][XS] updated actions (zero for state / unused rows)
  float* gain_s = xt + 8 * XS;                  // [128] final-norm gain of my channels
  float* bias_s = gain_s + 128;                 // [D] embedding bias
  float* gnext_s = bias_s + D;                  // [D] pi0.5: gain of layer 0's first norm
  float* ssw = gnext_s + D;                     // [16][8]
  float* wc_s = ssw + SB_WARPS * 8;             // [SB_MAXA][WS]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
  const int rank = (int)sb_cluster_rank();
  const int c0 = rank * 128;

  pdl_launch_dependents();
  unsigned long long* tr = (p.trace && tid == 0 && rank == 0) ? p.trace : nullptr;
  trace_stamp(tr, 0);
  // ---- ahead of the dependency wait: constants ---------------------------------------------------------------------
  if (tid == 0) {
    abort_flag = 0;
    recv_ok = 1;
    mbar_init(smem_u32(&bar_recv), 1);
    if (!p.first) mbar_expect_tx(smem_u32(&bar_recv), (uint32_t)(NC - 1) * PBYTES);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (!p.last) {
    // Wc -> shared memory (16-byte asynchronous copies, no registers), rows past the action width zero
    for (int i = tid; i < SB_MAXA * (D / 4); i += SB_THREADS) {
      const int a = i / (D / 4), c4 = i - a * (D / 4);
      const uint32_t dst = smem_u32(wc_s + a * WS + c4 * 4);
      if (a < A)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(p.Wc + (size_t)a * D + c4 * 4) : "memory");
      else
        *reinterpret_cast<float4*>(wc_s + a * WS + c4 * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    for (int i = tid; i < D; i += SB_THREADS) {
      bias_s[i] = __ldg(p.bias + i);
      gnext_s[i] = p.gain_next ? __ldg(p.gain_next + i) : 1.0f;
    }
  }
  // stage 1 B fragments: warp (mt, nt) multiplies token rows 16 mt .. + 15 by action channels 8 nt .. + 7
  const int mt1 = warp & 3, nt1 = warp >> 2;
  uint32_t bw[16][2];
  if (!p.first) {
    const int a = nt1 * 8 + g;
#pragma unroll
    for (int ks = 0; ks < 16; ++ks) {
      const int d = c0 + ks * 8 + t4;
      bw[ks][0] = a < A ? tf32_of(__ldg(p.Wout + (size_t)d * A + a)) : 0u;
      bw[ks][1] = a < A ? tf32_of(__ldg(p.Wout + (size_t)(d + 4) * A + a)) : 0u;
    }
    if (tid < 128) gain_s[tid] = __ldg(p.gain_f + c0 + tid);
    // shift term of my channels: sum_d shift[d] Wout[d][a], four d-ranges of 32 added in a fixed order
    if (tid < 128) {
      const int a2 = tid & 31, dq = tid >> 5;
      float q = 0.f;
      if (p.shift_f && a2 < A)
        for (int d = c0 + dq * 32; d < c0 + dq * 32 + 32; ++d) q = fmaf(__ldg(p.shift_f + d), __ldg(p.Wout + (size_t)d * A + a2), q);
      ssw[dq * 32 + a2] = q;
    }
  }
  // my rows: local row l (< 8) is token row 8 l + rank.  Thread (l = tid / 32, a = tid % 32) of the first eight warps
  // finishes element (l, a); lanes of the stage-2 epilogue handle row l = g.
  auto action_row = [&](int row) -> int {      // token row -> action row (or -1: a state token or past the end)
    if (row >= p.M) return -1;
    const int b = row / p.S, i = row - b * p.S;
    return i < p.ns ? -1 : b * p.H + i - p.ns;
  };
  const int my_r = tid < 256 ? action_row(8 * (tid >> 5) + rank) : -1;
  const float my_bout = (tid < 256 && lane < A && !p.first) ? __ldg(p.bout + lane) : 0.f;
  float* const xglob = p.rq->x;                   // (the request block is written before the captured loop starts)
  const int row2 = 8 * g + rank;                  // stage 2: the token row of this lane's accumulators
  const bool valid2 = row2 < p.M;
  const int b2 = valid2 ? row2 / p.S : 0;
  const bool state2 = valid2 && (row2 - b2 * p.S) < p.ns;
  for (int i = tid; i < 8 * XS; i += SB_THREADS) xt[i] = 0.f;
  __syncthreads();
  if (!p.first && tid < 32) {
    const float q = (ssw[tid] + ssw[32 + tid]) + (ssw[64 + tid] + ssw[96 + tid]);
#pragma unroll
    for (int c = 0; c < NC; ++c) part[c * PBLOCK + 8 * PS + tid] = q;
  }
  // every CTA's barrier exists before a peer can send to it
  sb_cluster_sync();
  trace_stamp(tr, 1);
  pdl_wait();
  trace_stamp(tr, 2);
  const bool store = !status_set(status);
  const WaitCtx wc{status, &abort_flag, p.wait_limit};

  if (!p.first) {
    // ---- stage 1: my channel slice of every row -> tf32(h * gain) in shared memory, the slice's sum of squares -------
    const float xold = (my_r >= 0 && lane < A) ? xglob[(size_t)my_r * A + lane] : 0.f;   // (needed after the exchange)
    {
      float4 v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int idx = tid + SB_THREADS * j, row = idx >> 5, c4 = idx & 31;
        v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row < p.M) v[j] = *reinterpret_cast<const float4*>(p.h_in + (size_t)row * D + c0 + c4 * 4);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int idx = tid + SB_THREADS * j, row = idx >> 5, c4 = idx & 31;
        const float ss = warp_sum(fmaf(v[j].x, v[j].x, fmaf(v[j].y, v[j].y, fmaf(v[j].z, v[j].z, v[j].w * v[j].w))));
        if (lane == 0) part[(row & 7) * PBLOCK + (row >> 3) * PS + 32] = ss;
        const float4 gn = *reinterpret_cast<const float4*>(gain_s + c4 * 4);
        float4 w;
        w.x = __uint_as_float(tf32_of(v[j].x * gn.x)), w.y = __uint_as_float(tf32_of(v[j].y * gn.y));
        w.z = __uint_as_float(tf32_of(v[j].z * gn.z)), w.w = __uint_as_float(tf32_of(v[j].w * gn.w));
        *reinterpret_cast<float4*>(h_s + row * HS + c4 * 4) = w;
      }
    }
    __syncthreads();
    trace_stamp(tr, 3);
    {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      const float* a_lo = h_s + (mt1 * 16 + g) * HS + t4;
      const float* a_hi = a_lo + 8 * HS;
#pragma unroll
      for (int ks = 0; ks < 16; ++ks)
        mma_tf32(acc, __float_as_uint(a_lo[ks * 8]), __float_as_uint(a_hi[ks * 8]), __float_as_uint(a_lo[ks * 8 + 4]),
                 __float_as_uint(a_hi[ks * 8 + 4]), bw[ks][0], bw[ks][1]);
      // rows 16 mt + g and + 8: same owner (row mod 8 = g), local rows 2 mt and 2 mt + 1
      float* o = part + g * PBLOCK + (2 * mt1) * PS + nt1 * 8 + 2 * t4;
      o[0] = acc[0], o[1] = acc[1], o[PS] = acc[2], o[PS + 1] = acc[3];
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the bulk-copy engine
    __syncthreads();
    trace_stamp(tr, 4);
    // ---- reduce-scatter by rows over the cluster ---------------------------------------------------------------------
    if (lane == 0 && warp < NC && warp != rank) {
      uint32_t dst, bar;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"(smem_u32(recv + rank * PBLOCK)), "r"(warp));
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar) : "r"(smem_u32(&bar_recv)), "r"(warp));
      asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                   "r"(smem_u32(part + warp * PBLOCK)), "r"(PBYTES), "r"(bar)
                   : "memory");
    }
    if (warp == 0) {
      const bool ok = mbar_wait_drain(smem_u32(&bar_recv), 0u, wc) > 0;
      if (lane == 0) recv_ok = ok ? 1 : 0;
    }
    __syncthreads();
    // what the peers sent has landed; they may leave once every CTA says the same (wait at the very end)
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    trace_stamp(tr, 5);
    // ---- my rows: the partials added in CTA order; Euler update --------------------------------------------------------
    if (my_r >= 0 && lane < A) {
      const int l = tid >> 5;
      float P = 0.f, ss = 0.f, Q = 0.f;
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const float* src = c == rank ? part + rank * PBLOCK : recv + c * PBLOCK;
        P += src[l * PS + lane], ss += src[l * PS + 32], Q += src[8 * PS + lane];
      }
      const float rs = rsqrtf(ss * (1.0f / (float)D) + p.eps);
      const float xn = xold + p.dt * (fmaf(rs, P, Q) + my_bout);
      xt[l * XS + lane] = xn;
      if (store && recv_ok && !*reinterpret_cast<volatile int*>(&abort_flag)) xglob[(size_t)my_r * A + lane] = xn;
    }
    trace_stamp(tr, 7);
    if (p.last) {
      asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
      return;
    }
  } else {
    if (my_r >= 0 && lane < A) xt[(tid >> 5) * XS + lane] = xglob[(size_t)my_r * A + lane];
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  trace_stamp(tr, 8);
  const bool good = store && recv_ok && !*reinterpret_cast<volatile int*>(&abort_flag);

  // ---- stage 2: my rows x channels 64 warp .. + 63, eight channels at a time (a rolled loop: this kernel runs once per
  // step, its instructions come from far away, so a short body matters more than instruction-level parallelism) --------
  {
    uint32_t af[4][2];
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) af[ks][0] = tf32_of(xt[g * XS + ks * 8 + t4]), af[ks][1] = tf32_of(xt[g * XS + ks * 8 + t4 + 4]);
    float ssl = 0.f;
#pragma unroll 1
    for (int nt = 0; nt < 8; ++nt) {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      const float* bp = wc_s + t4 * WS + warp * 64 + nt * 8 + g;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
        mma_tf32(acc, af[ks][0], 0u, af[ks][1], 0u, tf32_of(bp[ks * 8 * WS]), tf32_of(bp[(ks * 8 + 4) * WS]));
      const int ch = warp * 64 + nt * 8 + 2 * t4;
      const float2 bs = *reinterpret_cast<const float2*>(bias_s + ch);
      float v0 = acc[0] + bs.x, v1 = acc[1] + bs.y;
      // (row & 7 = rank: the swizzle term of the tiled layout is the same for all my rows)
      const size_t ti = ((size_t)(ch >> 6) * 64 + row2) * 64 + ((((ch & 63) >> 3) ^ rank) << 3) + (ch & 7);
      if (!p.ada) {
        v0 = state2 ? 0.f : __fdividef(v0, 1.0f + __expf(-v0)), v1 = state2 ? 0.f : __fdividef(v1, 1.0f + __expf(-v1));
        if (valid2 && good) *reinterpret_cast<__nv_bfloat162*>(p.u + ti) = __floats2bfloat162_rn(v0, v1);
      } else {
        if (state2) {
          const float2 s2 = __ldg(reinterpret_cast<const float2*>(p.state_tok + (size_t)b2 * D + ch));
          v0 = s2.x, v1 = s2.y;
        }
        if (valid2 && good) {
          const float2 gn = *reinterpret_cast<const float2*>(gnext_s + ch);
          *reinterpret_cast<float2*>(p.h_out + (size_t)row2 * D + ch) = make_float2(v0, v1);
          *reinterpret_cast<__nv_bfloat162*>(p.xn_out + ti) = __floats2bfloat162_rn(v0 * gn.x, v1 * gn.y);
        }
        ssl = fmaf(v0, v0, fmaf(v1, v1, ssl));
      }
    }
    if (p.ada) {
      // the warp's 64 channels of row g: the four lanes of a quad
      ssl += __shfl_xor_sync(0xffffffffu, ssl, 1);
      ssl += __shfl_xor_sync(0xffffffffu, ssl, 2);
      if (t4 == 0) ssw[warp * 8 + g] = ssl;
    }
  }
  trace_stamp(tr, 6);
  if (p.ada) {
    __syncthreads();
    // the row's whole sum of squares goes to slice 0 of the consumer's [8][64] table, zeros to the other slices
    if (tid < 64) {
      const int l = tid & 7, slice = tid >> 3, row = 8 * l + rank;
      float ss = 0.f;
      if (slice == 0)
#pragma unroll
        for (int w = 0; w < SB_WARPS; ++w) ss += ssw[w * 8 + l];
      if (row < p.M && good) p.ss_out[slice * 64 + row] = ss;
    }
  }
  if (!p.first) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

size_t step_b1_smem() {
  return ((size_t)64 * HS + 2 * SB_NC * PBLOCK + 8 * XS + 128 + 2 * SB_D + SB_WARPS * 8 + (size_t)SB_MAXA * WS) * sizeof(float);
}

}  // namespace

// Model width 1024 (8 slices of 128 channels), one 64-row token tile, an even action width of at most 32.
bool step_b1_supported(const Dims& d, int batch) {
  return d.D == SB_D && d.A <= SB_MAXA && d.A % 2 == 0 && batch * d.S <= 64;
}

cudaError_t launch_step_b1(int* status, const StepB1& p, cudaStream_t st) {
  static PerDeviceOnce once;
  if (once.needed()) {
    cudaError_t e = cudaFuncSetAttribute(k_step_b1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)step_b1_smem());
    if (e != cudaSuccess) return e;
    once.done();
  }
  cudaLaunchConfig_t cfg{};
  const int NC = SB_NC;
  cfg.gridDim = dim3(NC, 1, 1), cfg.blockDim = dim3(SB_THREADS), cfg.dynamicSmemBytes = step_b1_smem(), cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = NC, at[0].val.clusterDim.y = 1, at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at, cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, k_step_b1, status, p);
}

}  // namespace phyai
