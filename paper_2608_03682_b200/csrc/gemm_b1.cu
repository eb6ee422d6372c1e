// Cluster split-K GEMM for calls with a single 64-token tile (one request, or a few short ones).
//
// At this size every projection of a layer is a latency chain, not a throughput problem: 51 tokens against a
// 1024 x 2560 ... 4096 x 1024 weight matrix.  What costs time is (1) the number of dependent kernels per layer and
// (2) inside a kernel, the length of the k-loop of one CTA (each 64-wide k-step needs 8 KB of activations through
// the SM's L2 port and four N = 64 MMAs issued by one thread, ~0.18 us) and the epilogue of a whole 128 x 64 tile by
// one CTA.  So the work is cut the other way round:
//
//   * grid = (C k-ranges, N / 128 channel tiles); the C CTAs of a channel tile form a thread-block cluster.  A CTA
//     multiplies its 128 channels by its K / C slice: its weights (contiguous in the packed layout) are requested
//     before the programmatic dependency wait, its activations (contiguous in the 64-row tiled layout) right after,
//     all stages resident, no ring.
//   * the partial accumulators are reduced over distributed shared memory: every CTA stages its [token][128] fp32
//     partial in its own shared memory and pushes, with one bulk copy per peer, the token rows that peer owns;
//     owner c then holds C partials of its ~M / C tokens, adds them in rank order (bit-reproducible) and runs the
//     epilogue for those tokens only.  The epilogue is thereby spread over the cluster as well.
//   * the RMSNorm between two projections is folded into them: a residual projection's epilogue writes
//     h (fp32), bf16(h * gain_next) as the next projection's activation tile, and per (channel tile, token) the
//     partial sum of squares; the next projection multiplies its accumulator columns by
//     rsqrt(sum of the partials / D + eps) (the contraction is linear in that per-token factor) and adds, for
//     adaptive norms, the row shift . W from a per-step table.  No norm kernel, no slab-sum kernel.
//
// Epilogues: rotary QKV (rotated, scaled bf16 k / v rows, q as rows or as the cluster attention kernel's swizzled
// operand tiles), interleaved GeGLU (64 gate + 64 up channels per tile), gated residual with the next norm's
// operands (also: the second layer of the pi0 action / time MLP, bias and state-token rows instead of the residual).
// 512 threads: an epilogue is a chain of dependent instructions per thread, so items are small (four channels of a
// token) and the per-channel tables are read as 16-byte vectors.  Waits: see mbar_wait_drain -- a given-up
// wait suppresses the global stores but never the copy / reduce protocol, so peers are not left waiting and
// nothing is in flight at exit.
#include "kernels.h"
#include "ptx.cuh"
#include "tc.cuh"

namespace phyai {
namespace {

constexpr int W_BYTES = 128 * 128;     // one weight block: 128 out channels x 64 k (bf16)
constexpr int X_BYTES = 64 * 128;      // one activation block: 64 tokens x 64 k
constexpr int STAGE = W_BYTES + X_BYTES;
constexpr int MAXK = 8;                // k-steps per CTA, all resident (8 x 24 KB + the 32 KB receive area fit one SM)
constexpr int NT = 512, NW = NT / 32;   // threads / warps of a CTA: the epilogues are chains of dependent instructions per
                                        // thread, so more threads with less work each finish sooner
constexpr int ROWB = 128 * 4;          // one token row of a partial: 128 channels fp32
constexpr size_t B1_SMEM_MAX = 227 * 1024 - 2048;   // dynamic shared memory limit: the opt-in maximum less the static part
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ float4 lds4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Four e4m3 codes (one 32-bit word) -> two bf16 pairs, exactly, without the (slow-rate) conversion instructions.
// A code is S EEEE MMM (bias 7).  Its byte goes to the high byte of a 16-bit half (byte permute): the sign is then
// in place; the magnitude, moved down by four bits, puts EEEE into the low bits of bf16's exponent field and MMM
// at the top of its mantissa, i.e. the bf16 number 2^(E - 127) (1 + M/8) -- for E = 0 the bf16 subnormal
// 2^-126 (M/8).  One exact bf16x2 multiplication by 2^120 restores the bias: 2^(E - 7)(1 + M/8), and for E = 0
// 2^-6 (M/8), which is the value of e4m3's subnormals; zero stays zero.  (bf16 multiplication has no flush-to-zero
// mode: subnormal inputs are honoured.)  Five full-rate instructions per pair.
__device__ __forceinline__ void e4m3x4_to_bf16x4(uint32_t w, uint32_t& lo, uint32_t& hi) {
  uint32_t x0, x1;
  asm("prmt.b32 %0, %1, 0, 0x1404;" : "=r"(x0) : "r"(w));   // [b1 0 b0 0]
  asm("prmt.b32 %0, %1, 0, 0x3424;" : "=r"(x1) : "r"(w));   // [b3 0 b2 0]
  const uint32_t t0 = (x0 & 0x80008000u) | ((x0 >> 4) & 0x07F007F0u);
  const uint32_t t1 = (x1 & 0x80008000u) | ((x1 >> 4) & 0x07F007F0u);
  const uint32_t c = 0x7B807B80u;   // (2^120, 2^120)
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(lo) : "r"(t0), "r"(c));
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(hi) : "r"(t1), "r"(c));
}

// WB: bits per streamed weight -- 0 = the bf16 operand image itself, 8 = e4m3 codes, 4 = int4 codes; the codes are
// decoded to the bf16 image in shared memory ahead of the dependency wait.
template <int EPI, int WB>
__global__ void __launch_bounds__(NT, 1) k_gemm_b1(int* status, const B1Gemm g) {
  constexpr bool W8 = WB != 0;          // (weights arrive as codes)
  constexpr uint32_t CODE_BYTES = WB == 4 ? W_BYTES / 4 : W_BYTES / 2;   // one block of codes
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[MAXK];
  __shared__ __align__(8) uint64_t bar_w8[MAXK];       // e4m3 weights: the byte blocks have landed
  __shared__ __align__(8) uint64_t bar_accum, bar_recv;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag, suppress, acc_ok, recv_ok;
  __shared__ __align__(16) float rstd_tab[64], sc_tab[128], sh_tab[128];
  __shared__ int2 tok_tab[64];     // QKV: (rotary position, request * 64 + suffix row) of every token

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31, tid = threadIdx.x;
  const int C = (int)gridDim.x, rank = (int)cluster_rank(), tile = blockIdx.y;
  const int KC = g.K >> 6;
  const int kc_begin = (KC * rank) / C, nk = (KC * (rank + 1)) / C - kc_begin;
  const int M = g.M;
  const int tok_lo = (M * rank) / C, ntok = (M * (rank + 1)) / C - tok_lo;   // token rows this CTA reduces and finishes
  const int tpc_max = (64 + C - 1) / C;
  const uint32_t slot = (uint32_t)tpc_max * ROWB;

  pdl_launch_dependents();
  unsigned long long* tr = nullptr;
  if (g.trace && tid == 0) {
    if (g.trace_all) tr = g.trace + (size_t)(blockIdx.y * gridDim.x + blockIdx.x) * 16;   // every CTA, one slot each
    else if (blockIdx.x == 0 && blockIdx.y == 0) tr = g.trace;
  }
  trace_stamp(tr, 0);
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t region = (uint32_t)max(g.nk_max * STAGE, 64 * ROWB);
  const uint32_t stage = tiles;                        // [64 tokens][128] fp32 partial, over the consumed operand stages
  const uint32_t recv = tiles + region;                // [C sources][tpc_max][128] fp32
  const uint32_t rope_s = recv + (uint32_t)C * slot;   // QKV: [tpc_max tokens][64] (cos, sin) of this tile's channel pairs

  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < MAXK; ++s) mbar_init(smem_u32(&bar_full[s]), W8 ? 1 : 2), mbar_init(smem_u32(&bar_w8[s]), 1);
    mbar_init(smem_u32(&bar_accum), 1);
    mbar_init(smem_u32(&bar_recv), 1);
    if (C > 1 && ntok > 0) mbar_expect_tx(smem_u32(&bar_recv), (uint32_t)(C - 1) * (uint32_t)ntok * ROWB);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_slot), 64);
    tc_fence_before();
  }
  // every CTA's barriers exist before a peer can send to them (this is before the dependency wait)
  cluster_sync_all();
  trace_stamp(tr, 1);
  tc_fence_after();
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, *reinterpret_cast<volatile uint32_t*>(&tmem_slot), 0);
  const WaitCtx wc{status, &abort_flag, g.wait_limit};

  // ---- before the dependency wait: weights (constants) and per-channel constants ------------------------------
  if (lane == 0) {
    for (int s = warp; s < nk; s += NW) {
      if (W8) {
        // one byte (or half a byte) per weight: the 8 KB (4 KB) block of codes lands at the end of the stage's 16 KB
        // operand slot
        const uint32_t full = smem_u32(&bar_w8[s]);
        mbar_expect_tx(full, CODE_BYTES);
        bulk_g2s(tiles + (uint32_t)s * STAGE + W_BYTES - CODE_BYTES,
                 reinterpret_cast<const uint8_t*>(g.W8) + ((size_t)tile * KC + kc_begin + s) * CODE_BYTES, CODE_BYTES, full);
      } else {
        const uint32_t full = smem_u32(&bar_full[s]);
        mbar_expect_tx(full, W_BYTES);
        bulk_g2s(tiles + (uint32_t)s * STAGE, reinterpret_cast<const uint8_t*>(g.W) + ((size_t)tile * KC + kc_begin + s) * W_BYTES,
                 W_BYTES, full);
      }
    }
  }
  if (tid < 128) {
    const int n = tile * 128 + tid;
    float sc = 1.0f;
    if (EPI == B1_GEGLU) {
      const float* sp = tid >= 64 ? g.wscale2 : g.wscale;
      if (sp) sc = sp[tile * 64 + (tid & 63)];
    } else if (g.wscale) {
      sc = g.wscale[n];
    }
    sc_tab[tid] = sc;
    sh_tab[tid] = g.shift_row ? g.shift_row[n] : 0.0f;
  }
  float4 gate4 = make_float4(1.f, 1.f, 1.f, 1.f), gain4 = gate4;
  if (EPI == B1_RESID) {
    const int n = tile * 128 + lane * 4;
    if (g.gate) gate4 = __ldg(reinterpret_cast<const float4*>(g.gate + n));
    if (g.gain_next) gain4 = __ldg(reinterpret_cast<const float4*>(g.gain_next + n));
  }
  const int n0 = tile * 128;
  const int Nq = g.Hq * g.dh, Nk = g.Hkv * g.dh;
  const bool rot_tile = EPI == B1_QKV && n0 < Nq + Nk;
  if (EPI == B1_QKV) {
    // where every token sits (the request block is written before the captured loop starts: safe to read ahead of
    // the dependency wait), then the rotary rows of this CTA's tokens for the 64 channel pairs of this tile
    if (tid < 64) {
      int2 e = make_int2(0, 0);
      if (tid < M) {
        const int b = tid / g.S, i = tid - b * g.S;
        const int* cu = g.rq->cu_lens;
        e = make_int2(cu[b + 1] - cu[b] + g.koff + i, b * 64 + i);
      }
      tok_tab[tid] = e;
    }
    __syncthreads();
    if (rot_tile && g.rope) {
      const int nn = n0 < Nq ? n0 : n0 - Nq;
      const int t64 = (nn % g.dh) >> 7;
      for (int idx = tid; idx < ntok * 32; idx += NT) {
        const int tl = idx >> 5, c = idx & 31;
        const int pos = tok_tab[tok_lo + tl].x;
        const float4 v = __ldg(reinterpret_cast<const float4*>(g.rope + (size_t)pos * (g.dh >> 1) + t64 * 64) + c);
        asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(rope_s + (uint32_t)(tl * 32 + c) * 16), "f"(v.x), "f"(v.y),
                     "f"(v.z), "f"(v.w)
                     : "memory");
      }
    }
  }
  if (W8) {
    // codes -> bf16 in place, ahead of the dependency wait where the weights arrive early (they are constants), stage
    // by stage as the blocks land: warps 2 s and 2 s + 1 take stage s, 64 rows each (8 x 8 rows; a lane takes 16 codes
    // of a row and writes them as 32 bytes of the swizzled K-major bf16 image the MMA reads).  The codes sit at the end
    // of the image they expand into, so both warps of a stage read all their codes into registers, meet at a named
    // barrier, and only then write.  The per-channel scale stays in the epilogue.
    const int s = warp >> 1, hf = warp & 1;
    if (s < nk) {
      mbar_wait_drain(smem_u32(&bar_w8[s]), 0u, wc);
      const uint32_t slot0 = tiles + (uint32_t)s * STAGE;
      const int r0 = hf * 64 + (lane >> 2), cq = lane & 3;       // my row of every group of 8 rows, my quarter of a row
      if constexpr (WB == 8) {
        uint4 raw[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t src = slot0 + W_BYTES - CODE_BYTES + (uint32_t)(r0 + 8 * j) * 64 + (uint32_t)cq * 16;
          asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(raw[j].x), "=r"(raw[j].y), "=r"(raw[j].z), "=r"(raw[j].w) : "r"(src) : "memory");
        }
        asm volatile("bar.sync %0, 64;" ::"r"(1 + s) : "memory");
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int r = r0 + 8 * j;
          const uint32_t words[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
#pragma unroll
          for (int c = 0; c < 2; ++c) {       // 16-byte chunk 2 cq + c of the row: 8 codes = words[2c], words[2c + 1]
            uint32_t o0, o1, o2, o3;
            e4m3x4_to_bf16x4(words[2 * c], o0, o1);
            e4m3x4_to_bf16x4(words[2 * c + 1], o2, o3);
            const uint32_t dst = slot0 + (uint32_t)r * 128 + (uint32_t)((((2 * cq + c) ^ (r & 7))) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
          }
        }
      } else {
        // int4: a row of the block is 32 bytes = 64 codes, byte j = codes (k = 2j in the low nibble, 2j + 1 in the
        // high one).  A nibble c becomes the bf16 number 128 + c by bit insertion (0x4300 | c: the unit of the mantissa
        // at 128 is 1), and one exact bf16x2 subtraction of 136 makes it c - 8.
        uint2 raw[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t src = slot0 + W_BYTES - CODE_BYTES + (uint32_t)(r0 + 8 * j) * 32 + (uint32_t)cq * 8;
          asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(raw[j].x), "=r"(raw[j].y) : "r"(src) : "memory");
        }
        asm volatile("bar.sync %0, 64;" ::"r"(1 + s) : "memory");
        auto pair = [](uint32_t byte) -> uint32_t {       // one byte -> (bf16(lo - 8), bf16(hi - 8))
          uint32_t w = 0x43004300u | (byte & 15u) | ((byte & 0xF0u) << 12), o;
          asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(o) : "r"(w), "r"(0x43084308u));
          return o;
        };
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int r = r0 + 8 * j;
          const uint32_t words[2] = {raw[j].x, raw[j].y};
#pragma unroll
          for (int c = 0; c < 2; ++c) {       // 16-byte chunk 2 cq + c: codes of bytes 4c .. 4c + 3 of my 8
            const uint32_t w4 = words[c];
            const uint32_t dst = slot0 + (uint32_t)r * 128 + (uint32_t)((((2 * cq + c) ^ (r & 7))) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(pair(w4 & 0xFFu)), "r"(pair((w4 >> 8) & 0xFFu)),
                         "r"(pair((w4 >> 16) & 0xFFu)), "r"(pair(w4 >> 24))
                         : "memory");
          }
        }
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the tensor core's reads
    __syncthreads();
    trace_stamp(tr, 10);
  }
  pdl_wait();
  trace_stamp(tr, 2);
  // ---- after it: activations, the status word, per-token factors (nothing the MMA warp has to wait for) -----------
  if (lane == 0) {
    for (int s = (warp + 4) & (NW - 1); s < nk; s += NW) {
      const uint32_t full = smem_u32(&bar_full[s]);
      mbar_expect_tx(full, X_BYTES);
      bulk_g2s(tiles + (uint32_t)s * STAGE + W_BYTES, reinterpret_cast<const uint8_t*>(g.X) + (size_t)(kc_begin + s) * X_BYTES,
               X_BYTES, full);
    }
  }
  float4 hpre[2];
  // B1_RESID: what the projection output is added to -- the residual stream, or (MLP second layer) the bias / the state
  // token's embedding
  auto is_state_row = [&](int tok) -> bool { return g.bias && (tok % g.S) < g.ns; };
  auto old_of = [&](int tok) -> float4 {
    const int n = tile * 128 + lane * 4;
    if (g.bias) {
      const int b = tok / g.S;
      return (tok - b * g.S) < g.ns ? __ldg(reinterpret_cast<const float4*>(g.state_tok + (size_t)b * g.N + n))
                                    : __ldg(reinterpret_cast<const float4*>(g.bias + n));
    }
    return *reinterpret_cast<const float4*>(g.h + (size_t)tok * g.ldh + n);
  };
  if (warp != 1) {
    if (tid == NT - 1) suppress = status_set(status) ? 1 : 0;
    if (tid >= 64 && tid < 128) {
      const int t = tid - 64;
      float r = 1.0f;
      if (g.ss_part && t < M) {
        float ss = 0.f;
        for (int i = 0; i < g.ss_n; ++i) ss += g.ss_part[i * 64 + t];
        r = 1.0f / sqrtf(ss * g.inv_D + g.eps);
      }
      rstd_tab[t] = r;
    }
  }
  if (EPI == B1_RESID) {
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int tl = warp + NW * u;
      hpre[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (tl < ntok) hpre[u] = old_of(tok_lo + tl);
    }
  }

  // ---- MMAs: one warp, whole warp in the loop, one elected lane issues -----------------------------------------
  if (warp == 1) {
    bool all_ok = true;
    for (int s = 0; s < nk; ++s) {
      const bool ok = mbar_wait_drain(smem_u32(&bar_full[s]), 0u, wc) > 0;
      all_ok = all_ok && ok;
      const uint32_t a0 = tiles + (uint32_t)s * STAGE;
      const uint64_t da = make_desc(a0), db = make_desc(a0 + W_BYTES);
      if (__all_sync(0xffffffffu, ok)) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (elect_one()) umma_bf16(tmem_base, da + 2 * k, db + 2 * k, IDESC, (s > 0 || k > 0) ? 1u : 0u);
      }
      __syncwarp();
    }
    if (elect_one()) umma_commit(smem_u32(&bar_accum));
    __syncwarp();
    const bool okc = mbar_wait_drain(smem_u32(&bar_accum), 0u, wc) > 0;
    if (lane == 0) acc_ok = (all_ok && okc && nk > 0) ? 1 : 0;
  }
  __syncthreads();
  tc_fence_after();
  trace_stamp(tr, 3);

  // ---- accumulator -> staging [token][channel] (the operand stages are free: every MMA has completed) -------------
  {
    // warp (q, cg): TMEM lanes 32 q .. + 31 (channels), columns 16 cg .. + 15 (tokens)
    const int q = warp & 3, cg = warp >> 2;
    if (cg * 16 < M) {
      float v[16];
      if (nk > 0) {
        tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(cg * 16), v);
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = 0.f;
      }
      const uint32_t dst = stage + (uint32_t)(cg * 16) * ROWB + (uint32_t)(q * 32 + lane) * 4;
#pragma unroll
      for (int j = 0; j < 16; ++j)
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(dst + (uint32_t)j * ROWB), "f"(v[j]) : "memory");
    }
  }
  tc_fence_before();
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the bulk-copy engine
  __syncthreads();
  // ---- reduce-scatter over the cluster: every peer gets its token rows of my partial -----------------------------
  // (one copy per warp: the bulk copies issued by one warp complete one after the other)
  if (lane == 0 && warp < C && warp != rank) {
    const int lo = (M * warp) / C, n = (M * (warp + 1)) / C - lo;
    if (n > 0) {
      uint32_t dst, bar;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"(recv + (uint32_t)rank * slot), "r"(warp));
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar) : "r"(smem_u32(&bar_recv)), "r"(warp));
      asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                   "r"(stage + (uint32_t)lo * ROWB), "r"((uint32_t)n * ROWB), "r"(bar)
                   : "memory");
    }
  }
  if (warp == 0) {
    bool ok = true;
    if (C > 1 && ntok > 0) ok = mbar_wait_drain(smem_u32(&bar_recv), 0u, wc) > 0;
    if (lane == 0) recv_ok = ok ? 1 : 0;
  }
  __syncthreads();
  // From here on this CTA no longer needs its peers: what they sent has landed.  It may leave once every peer says the
  // same (then every copy out of its own staging area has completed): arrive now, wait at the very end, so that the
  // skew between the CTAs hides behind the epilogue.
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  trace_stamp(tr, 4);
  const bool store = !suppress && acc_ok && recv_ok && !*reinterpret_cast<volatile int*>(&abort_flag);

  // four consecutive channels of one of my tokens: the C partials added in rank order
  auto sum4 = [&](int tl, int ch) -> float4 {
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c = 0; c < C; ++c) {
      const uint32_t p = (c == rank) ? stage + (uint32_t)(tok_lo + tl) * ROWB : recv + (uint32_t)c * slot + (uint32_t)tl * ROWB;
      const float4 v = lds4(p + (uint32_t)ch * 4);
      a.x += v.x, a.y += v.y, a.z += v.z, a.w += v.w;
    }
    return a;
  };
  // accumulator value -> projection output: weight scale, the folded norm's per-token factor, the folded shift row
  // (four consecutive channels at a time: the tables are read as 16-byte vectors; no shift table without a shift)
  const bool has_shift = g.shift_row != nullptr;
  auto fin4 = [&](float4 x, int ch, float r) -> float4 {
    const float4 s0 = *reinterpret_cast<const float4*>(sc_tab + ch);
    float4 h0 = make_float4(0.f, 0.f, 0.f, 0.f);
    if (has_shift) h0 = *reinterpret_cast<const float4*>(sh_tab + ch);
    return make_float4(fmaf(x.x * s0.x, r, h0.x), fmaf(x.y * s0.y, r, h0.y), fmaf(x.z * s0.z, r, h0.z), fmaf(x.w * s0.w, r, h0.w));
  };

  if (store) {
    if (EPI == B1_QKV) {
      if (rot_tile) {
        const bool isq = n0 < Nq;
        const int nn = isq ? n0 : n0 - Nq;
        const int head = nn / g.dh, t64 = (nn - head * g.dh) >> 7, half = g.dh >> 1;
        __nv_bfloat16* base = isq ? g.qr : g.kr;
        const int H = isq ? g.Hq : g.Hkv;
        const float osc = isq ? rsqrtf((float)g.dh) : 1.0f;
        // an item: four channels of the head's first half and their four rotary partners, of one token
        for (int it = tid; it < ntok * 16; it += NT) {
          const int tl = it >> 4, j0 = (it & 15) * 4;
          const int2 e = tok_tab[tok_lo + tl];
          const float r = rstd_tab[tok_lo + tl];
          float4 lo = fin4(sum4(tl, j0), j0, r), hi = fin4(sum4(tl, 64 + j0), 64 + j0, r);
          if (g.rope) {
            const float4 c0 = lds4(rope_s + (uint32_t)(tl * 64 + j0) * 8);       // (cos, sin) of channels j0, j0 + 1
            const float4 c1 = lds4(rope_s + (uint32_t)(tl * 64 + j0 + 2) * 8);   // ... j0 + 2, j0 + 3
            const float4 l = lo, h = hi;
            lo.x = l.x * c0.x - h.x * c0.y, hi.x = h.x * c0.x + l.x * c0.y;
            lo.y = l.y * c0.z - h.y * c0.w, hi.y = h.y * c0.z + l.y * c0.w;
            lo.z = l.z * c1.x - h.z * c1.y, hi.z = h.z * c1.x + l.z * c1.y;
            lo.w = l.w * c1.z - h.w * c1.w, hi.w = h.w * c1.z + l.w * c1.w;
          }
          const int b = e.y >> 6, i = e.y & 63;
          const uint2 vlo = make_uint2(pack2(lo.x * osc, lo.y * osc), pack2(lo.z * osc, lo.w * osc));
          const uint2 vhi = make_uint2(pack2(hi.x * osc, hi.y * osc), pack2(hi.z * osc, hi.w * osc));
          if (isq && g.q_tiles) {
            // q as the attention kernel's operand tiles: per (request, head pair) dh / 64 blocks of [128 rows][64
            // channels], row = 64 * (head & 1) + token, the 16-byte chunks of a 128-byte row XOR-swizzled by row & 7
            const int rw = (head & 1) * 64 + i, c_lo = t64 * 64 + j0, c_hi = c_lo + half;
            __nv_bfloat16* tb = g.q_tiles + (size_t)(b * (g.Hq >> 1) + (head >> 1)) * (size_t)(128 * g.dh);
            *reinterpret_cast<uint2*>(tb + (size_t)(c_lo >> 6) * 8192 + rw * 64 + ((((c_lo & 63) >> 3) ^ (rw & 7)) << 3) + (c_lo & 7)) = vlo;
            *reinterpret_cast<uint2*>(tb + (size_t)(c_hi >> 6) * 8192 + rw * 64 + ((((c_hi & 63) >> 3) ^ (rw & 7)) << 3) + (c_hi & 7)) = vhi;
          } else {
            // (q: one row per query token; k: the request's key rows, query row i at key row koff + i)
            __nv_bfloat16* dst = base + (isq ? ((size_t)(b * H + head) * g.S + i) : ((size_t)(b * H + head) * g.Sk_stride + g.koff + i)) * g.dh +
                                 t64 * 64 + j0;
            *reinterpret_cast<uint2*>(dst) = vlo;
            *reinterpret_cast<uint2*>(dst + half) = vhi;
          }
        }
      } else {
        const int nn = n0 - Nq - Nk;
        const int head = nn / g.dh, coff = nn - head * g.dh;       // 128 consecutive v channels
        for (int it = tid; it < ntok * 32; it += NT) {
          const int tl = it >> 5, j0 = (it & 31) * 4;
          const int2 e = tok_tab[tok_lo + tl];
          const float4 x = fin4(sum4(tl, j0), j0, rstd_tab[tok_lo + tl]);
          const int b = e.y >> 6, i = e.y & 63;
          *reinterpret_cast<uint2*>(g.vr + ((size_t)(b * g.Hkv + head) * g.Sk_stride + g.koff + i) * g.dh + coff + j0) =
              make_uint2(pack2(x.x, x.y), pack2(x.z, x.w));
        }
      }
    } else if (EPI == B1_GEGLU) {
      // rows 0..63 = gate channels f0 .. f0 + 63, rows 64..127 = the matching up channels; the result is one 64-wide
      // k-chunk (`tile`) of the down projection's activation tile, written as halves of its swizzled 16-byte groups
      for (int it = tid; it < ntok * 16; it += NT) {
        const int tl = it >> 4, c4 = it & 15, j0 = c4 * 4, tok = tok_lo + tl;
        const float r = rstd_tab[tok];
        const float4 gt = fin4(sum4(tl, j0), j0, r), up = fin4(sum4(tl, 64 + j0), 64 + j0, r);
        const float m0 = gelu_fast(gt.x, g.gelu_exact) * up.x, m1 = gelu_fast(gt.y, g.gelu_exact) * up.y;
        const float m2 = gelu_fast(gt.z, g.gelu_exact) * up.z, m3 = gelu_fast(gt.w, g.gelu_exact) * up.w;
        *reinterpret_cast<uint2*>(g.out_tiled + ((size_t)tile * 64 + tok) * 64 + (((c4 >> 1) ^ (tok & 7)) << 3) + (c4 & 1) * 4) =
            make_uint2(pack2(m0, m1), pack2(m2, m3));
      }
    } else {
      // gated residual: one warp per token, a lane takes four channels.  h stays fp32; the next projection's
      // activation tile is bf16(h * gain) (its 1 / rms factor follows in that projection's epilogue from the
      // partial sums of squares written here)
      auto token = [&](int tl, bool have_old, float4 old) {
        const int tok = tok_lo + tl, n = n0 + lane * 4;
        float* hp = g.h + (size_t)tok * g.ldh + n;
        if (!have_old) old = old_of(tok);
        float4 a = sum4(tl, lane * 4);
        if (is_state_row(tok)) a = make_float4(0.f, 0.f, 0.f, 0.f);
        float4 hv;
        const float4 sc = *reinterpret_cast<const float4*>(sc_tab + lane * 4);
        hv.x = old.x + gate4.x * (a.x * sc.x), hv.y = old.y + gate4.y * (a.y * sc.y);
        hv.z = old.z + gate4.z * (a.z * sc.z), hv.w = old.w + gate4.w * (a.w * sc.w);
        *reinterpret_cast<float4*>(hp) = hv;
        if (g.xn_out) {
          *reinterpret_cast<uint2*>(g.xn_out + tiled_index(tok, n, 64)) =
              make_uint2(pack2(hv.x * gain4.x, hv.y * gain4.y), pack2(hv.z * gain4.z, hv.w * gain4.w));
          const float ss = warp_sum(hv.x * hv.x + hv.y * hv.y + hv.z * hv.z + hv.w * hv.w);
          if (lane == 0) g.ss_out[tile * 64 + tok] = ss;
        }
      };
      if (warp < ntok) token(warp, true, hpre[0]);           // (the first two rows of a warp were requested early)
      if (warp + NW < ntok) token(warp + NW, true, hpre[1]);
      for (int tl = warp + 2 * NW; tl < ntok; tl += NW) token(tl, false, make_float4(0.f, 0.f, 0.f, 0.f));
    }
  }
  trace_stamp(tr, 5);
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  trace_stamp(tr, 6);
  if (tr) {
    unsigned sm;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
    tr[7] = sm;
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 64);
  }
}

size_t b1_smem(int nk_max, int C, bool rope_rows) {
  const int tpc = (64 + C - 1) / C;
  const size_t region = (size_t)(nk_max * STAGE > 64 * ROWB ? nk_max * STAGE : 64 * ROWB);
  return 1024 + region + (size_t)C * tpc * ROWB + (rope_rows ? (size_t)tpc * 512 : 0);
}

template <int EPI, int WB>
cudaError_t launch_one(int* status, const B1Gemm& g, int C, cudaStream_t st) {
  static PerDeviceOnce once;
  if (once.needed()) {
    cudaError_t e = cudaFuncSetAttribute(k_gemm_b1<EPI, WB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)B1_SMEM_MAX);
    if (e != cudaSuccess) return e;
    once.done();
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(C, g.N / 128, 1), cfg.blockDim = dim3(NT), cfg.dynamicSmemBytes = b1_smem(g.nk_max, C, g.epi == B1_QKV), cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = C, at[0].val.clusterDim.y = 1, at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at, cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, k_gemm_b1<EPI, WB>, status, g);
}

}  // namespace

// Largest cluster size (k-ranges per channel tile) for a projection with `tiles` channel tiles and KC k-chunks:
// at most 8 (portable cluster size), at most one CTA per SM in total, at most one k-chunk per CTA.
int b1_pick_cluster(int tiles, int KC, int n_sm) {
  int C = n_sm / tiles;
  if (C > 8) C = 8;
  if (C > KC) C = KC;
  if (C < 1) C = 1;
  return C;
}
// A projection fits when its k-steps per CTA stay resident (<= MAXK) and the cluster has at most one CTA per SM.
bool b1_gemm_supported(int N, int K, int C, int n_sm, bool qkv) {
  if (N % 128 || K % 64 || C < 1 || C > 8 || C > K / 64) return false;
  if ((N / 128) * C > 2 * n_sm) return false;
  const int nk = (K / 64 + C - 1) / C;
  return nk <= MAXK && b1_smem(nk, C, qkv) <= B1_SMEM_MAX;
}

cudaError_t launch_b1_gemm(int* status, const B1Gemm& g_in, int C, cudaStream_t st) {
  B1Gemm g = g_in;
  const int KC = g.K / 64;
  g.nk_max = (KC + C - 1) / C;
  if (b1_smem(g.nk_max, C, g.epi == B1_QKV) > B1_SMEM_MAX) return cudaErrorInvalidConfiguration;
  if (g.W8 && g.w_bits == 4) {
    if (g.epi == B1_QKV) return launch_one<B1_QKV, 4>(status, g, C, st);
    if (g.epi == B1_GEGLU) return launch_one<B1_GEGLU, 4>(status, g, C, st);
    return launch_one<B1_RESID, 4>(status, g, C, st);
  }
  if (g.W8) {
    if (g.epi == B1_QKV) return launch_one<B1_QKV, 8>(status, g, C, st);
    if (g.epi == B1_GEGLU) return launch_one<B1_GEGLU, 8>(status, g, C, st);
    return launch_one<B1_RESID, 8>(status, g, C, st);
  }
  if (g.epi == B1_QKV) return launch_one<B1_QKV, 0>(status, g, C, st);
  if (g.epi == B1_GEGLU) return launch_one<B1_GEGLU, 0>(status, g, C, st);
  return launch_one<B1_RESID, 0>(status, g, C, st);
}

}  // namespace phyai
