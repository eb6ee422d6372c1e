// Persistent tile GEMM for many token tiles: one CTA per SM walks over 128-row x 256-token output tiles, and the
// epilogue of one tile runs while the tensor cores work on the next.  Two epilogues: the gate / up projection with
// GeGLU (the expert MLP's first layer, m = gelu(x Wg) * (x Wu)) and the fused q | k | v projection with the rotary
// embedding (the attention kernel's operands, bf16).
//
// Why a kernel of its own.  With one 256-token x 256-row tile per CTA (two accumulators of 128 rows) the 512
// tensor-memory columns are full, so a tile's epilogue (3.5 - 5 us of fp32 work for 65536 accumulator values, 8 - 12 us
// on the first CTA of an SM while the code is fetched) cannot overlap anything: measured per tile of the gate / up
// projection 9.9 us of main loop, 5 - 11 us of epilogue, ~2.5 us of launch / set-up / first operands, i.e. the tensor
// pipe idles half the time.  Here a tile is 128 weight rows x 256 tokens (256 columns), two accumulators alternate, and
// the weight rows are interleaved so that the two rows which the epilogue combines sit in one warp's tensor-memory
// lanes i and i + 16: rows 32 q + i (i < 16) are the gate rows (q / k: the first-half channels) of 16 channels, rows
// 32 q + 16 + i the up rows (the rotary partners) of the same channels.  They meet through one warp shuffle and the
// result goes straight to global memory: no shared-memory staging, no barrier among the epilogue warps (q | k | v: one
// per tile, for the token table), and the operand stages stay with the main loop.
// The price is 48 KB instead of 64 KB of operands per (128 x 256 x 64) MACs x 2, i.e. 1.5 x the bytes per flop: the
// main loop runs at the SM's ingest rate (measured 62 bytes per clock with all SMs streaming), ~6.4 us per tile at
// K = 1024, which still beats 17 - 24 us per pair of such tiles.
//
// Roles (800 threads): warps 0-7 issue bulk copies (one weight block of 16 KB and two activation pieces of 16 KB per
// k-chunk, four stages), warp 8 issues the MMAs, warps 9-24 are the epilogue (tensor-memory lane quarter = warp % 4,
// 64 of the 256 token columns each).  Every wait is bounded; after a give-up the pipeline keeps running (copies,
// commits, barriers) with MMAs and stores skipped, so nothing is in flight when the CTA exits.
#include "kernels.h"
#include "ptx.cuh"
#include "tc.cuh"

namespace phyai {
namespace {

constexpr int GU_NT = 256;                  // tokens per tile
constexpr int BAR_PEPI = 1, NPEPI = 512;    // named barrier of the 16 epilogue warps
constexpr int GU_STAGES = 4;
constexpr int GU_A_BYTES = 128 * 128;       // weight block: 128 rows x 128 bytes
constexpr int GU_B_PIECE = 128 * 128;       // activation piece: 128 tokens x 128 bytes
constexpr int GU_NCOPY = 3;
constexpr int GU_STAGE_BYTES = GU_A_BYTES + 2 * GU_B_PIECE;
constexpr int GU_NPROD = 8;
constexpr size_t GU_SMEM = (size_t)GU_STAGES * GU_STAGE_BYTES + 1024;
static_assert((GU_NPROD + GU_NCOPY - 1) / GU_NCOPY <= GU_STAGES, "producer stride exceeds the stage ring");

template <bool F8, bool QKV>
__global__ void __launch_bounds__(800, 1) k_gemm_persist(int* status, const PersistGemm g) {
  // instruction descriptors: D fp32 (bit 4), A / B bf16 (bits 7, 10) or e4m3 (format fields 0), K-major, N >> 3 at
  // bit 17, M >> 4 at bit 24
  constexpr uint32_t IDESC = F8 ? ((1u << 4) | ((uint32_t)(GU_NT >> 3) << 17) | ((128u >> 4) << 24))
                                : ((1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(GU_NT >> 3) << 17) | ((128u >> 4) << 24));
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[GU_STAGES];
  __shared__ __align__(8) uint64_t bar_empty[GU_STAGES];
  __shared__ __align__(8) uint64_t bar_tfull[2];    // accumulator complete (MMA commit)
  __shared__ __align__(8) uint64_t bar_tempty[2];   // accumulator read out (16 epilogue warps)
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int skip_flag;
  // q | k | v: per token (position x dh / 2, element offset of its row in q [b][Hq][S][dh] without the head term, the
  // same for k / v [b][Hkv][S][dh], 1 if the token exists)
  __shared__ int4 tok_tab[QKV ? 2 : 1][QKV ? GU_NT : 1];

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const int KC = F8 ? g.K >> 7 : g.K >> 6;         // k-chunks of 128 bytes per operand row
  const int n_n = g.N >> 7;                        // weight tiles of 128 packed rows
  const int n_t = (g.M + GU_NT - 1) / GU_NT;       // token tiles
  const int n_tiles = n_n * n_t;
  const int n_my = ((int)blockIdx.x < n_tiles) ? (n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const int steps = n_my * KC;                     // k-steps of this CTA over all its tiles

  pdl_launch_dependents();
  unsigned long long* const trc = g.trace ? g.trace + (size_t)blockIdx.x * 16 : nullptr;
  if (threadIdx.x == 0) trace_stamp(trc, 0);
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < GU_STAGES; ++s) {
      mbar_init(smem_u32(&bar_full[s]), GU_NCOPY);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bar_tfull[b]), 1);
      mbar_init(smem_u32(&bar_tempty[b]), 16);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    tmem_alloc(smem_u32(&tmem_slot), 512);
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  if (threadIdx.x == 0) trace_stamp(trc, 1);
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, *reinterpret_cast<volatile uint32_t*>(&tmem_slot), 0);
  const WaitCtx wc{status, &abort_flag, g.wait_limit};

  // k-step gi of this CTA: tile (gi / KC) of its list, k-chunk gi % KC
  auto w_src = [&](int gi) -> const uint8_t* {
    const int t = (int)blockIdx.x + (gi / KC) * (int)gridDim.x;
    return reinterpret_cast<const uint8_t*>(g.W) + ((size_t)(t % n_n) * KC + gi % KC) * GU_A_BYTES;
  };
  auto x_src = [&](int gi, int pc) -> const uint8_t* {
    const int t = (int)blockIdx.x + (gi / KC) * (int)gridDim.x;
    return reinterpret_cast<const uint8_t*>(g.X) + ((size_t)(gi % KC) * g.rows_pad + (size_t)(t / n_n) * GU_NT) * 128 +
           (size_t)pc * GU_B_PIECE;
  };
  auto issue = [&](int gi, int c) {
    const uint32_t s = (uint32_t)(gi % GU_STAGES);
    const uint32_t full = smem_u32(&bar_full[s]);
    const uint32_t dst = tiles + s * GU_STAGE_BYTES;
    if (c == 0) {
      mbar_expect_tx(full, GU_A_BYTES);
      bulk_g2s(dst, w_src(gi), GU_A_BYTES, full);
    } else {
      mbar_expect_tx(full, GU_B_PIECE);
      bulk_g2s(dst + GU_A_BYTES + (c - 1) * GU_B_PIECE, x_src(gi, c - 1), GU_B_PIECE, full);
    }
  };
  // Programmatic dependent launch: the weight blocks of the first stages are on their way before the kernel that
  // produces the activations has finished.
  const int n_early = steps < GU_STAGES ? steps : GU_STAGES;
  const bool issues = lane == 0 && warp < GU_NPROD;
  if (issues)
    for (int id = warp; id < n_early * GU_NCOPY; id += GU_NPROD)
      if (id % GU_NCOPY == 0) issue(id / GU_NCOPY, 0);
  pdl_wait();
  if (threadIdx.x == 0) trace_stamp(trc, 2);
  // (the activation copies of those stages go out before the status word is known: the skip path waits for them)
  if (issues)
    for (int id = warp; id < n_early * GU_NCOPY; id += GU_NPROD)
      if (id % GU_NCOPY != 0) issue(id / GU_NCOPY, id % GU_NCOPY);
  if (threadIdx.x == GU_NPROD * 32) skip_flag = status_set(status) || steps <= 0;
  __syncthreads();
  if (skip_flag) {
    if (threadIdx.x == 0)
      for (int i = 0; i < n_early; ++i) mbar_wait_drain(smem_u32(&bar_full[i]), 0u, wc);
    __syncthreads();
    if (warp == 8) {
      tc_fence_after();
      tmem_dealloc(tmem_base, 512);
    }
    return;
  }

  if (warp < GU_NPROD) {
    // ---------------- copy issuers: copy number id = k-step * 3 + piece goes to warp id % 8 ----------------------
    if (lane == 0) {
      for (int id = warp + (n_early * GU_NCOPY - warp + GU_NPROD - 1) / GU_NPROD * GU_NPROD; id < steps * GU_NCOPY;
           id += GU_NPROD) {
        const int gi = id / GU_NCOPY;
        const uint32_t ph = (uint32_t)(gi / GU_STAGES) & 1u;
        if (mbar_wait_drain(smem_u32(&bar_empty[gi % GU_STAGES]), ph ^ 1u, wc) < 0) break;
        issue(gi, id % GU_NCOPY);
      }
    }
  } else if (warp == 8) {
    // ---------------- MMA issuer (whole warp in the loop, one elected lane issues) --------------------------------
    int gi = 0;
    bool dead = false;
    for (int i = 0; i < n_my && !dead; ++i) {
      const int buf = i & 1;
      // the epilogue has read the accumulator that this tile overwrites (two tiles ago)
      bool ok = mbar_wait_drain(smem_u32(&bar_tempty[buf]), (((uint32_t)i >> 1) & 1u) ^ 1u, wc) > 0;
      tc_fence_after();
      const uint32_t tacc = tmem_base + (uint32_t)buf * GU_NT;
      for (int k = 0; k < KC; ++k, ++gi) {
        const int s = gi % GU_STAGES;
        const uint32_t ph = (uint32_t)(gi / GU_STAGES) & 1u;
        const int r = mbar_wait_drain(smem_u32(&bar_full[s]), ph, wc);
        if (gi == 0 && lane == 0) trace_stamp(trc, 3);
        if (r < 0) {
          dead = true;   // (copies that never landed: nothing more can be done with this pipeline)
          break;
        }
        ok = ok && r > 0;
        const uint32_t a0 = tiles + (uint32_t)s * GU_STAGE_BYTES;
        const uint64_t da = make_desc(a0), db = make_desc(a0 + GU_A_BYTES);
        if (__all_sync(0xffffffffu, ok)) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {   // 4 MMAs of 32 bytes of k per 128-byte chunk: +2 descriptor units each
            const uint32_t acc = (k > 0 || kk > 0) ? 1u : 0u;
            if constexpr (F8) {
              if (elect_one()) umma_f8(tacc, da + 2 * kk, db + 2 * kk, IDESC, acc);
            } else {
              if (elect_one()) umma_bf16(tacc, da + 2 * kk, db + 2 * kk, IDESC, acc);
            }
          }
        }
        if (gi + GU_STAGES < steps && elect_one()) umma_commit(smem_u32(&bar_empty[s]));
        __syncwarp();
      }
      if (!dead && elect_one()) umma_commit(smem_u32(&bar_tfull[buf]));
      __syncwarp();
    }
    if (lane == 0) trace_stamp(trc, 4);
  } else {
    // ---------------- epilogue: tensor memory -> registers -> global ---------------------------------------------
    const int ew = warp - 9;                 // 0..15
    const int q = warp & 3, hf = ew >> 2;    // tensor-memory lane quarter, quarter of the token columns
    const int hi = lane >> 4;                // 0: this lane holds a gate / first-half row, 1: an up / partner row
    const int cl = 16 * q + (lane & 15);     // channel within the tile's 64
    const int et = ew * 32 + lane;
    bool dead = false;
    for (int i = 0; i < n_my; ++i) {
      const int buf = i & 1;
      const int t = (int)blockIdx.x + i * (int)gridDim.x;
      const int nt = t % n_n, tok_base = (t / n_n) * GU_NT;
      // (per-row weight scales of the tile and, q | k | v, the token table: before the accumulator is complete)
      float s_lo = 1.0f, s_hi = 1.0f;
      if constexpr (QKV) {
        // packed row of this lane's channel and of its partner in the scale vector's (un-interleaved) order
        if (g.scale_g) s_lo = g.scale_g[nt * 128 + cl], s_hi = g.scale_g[nt * 128 + 64 + cl];
        if (et < GU_NT) {
          const int tok = tok_base + et;
          int4 e = make_int4(0, 0, 0, 0);
          if (tok < g.M) {
            const int b = tok / g.S, ii = tok - b * g.S;
            const int* cu = g.rq->cu_lens;
            e = make_int4((cu[b + 1] - cu[b] + ii) * (g.dh >> 1), (b * g.Hq * g.S + ii) * g.dh, (b * g.Hkv * g.S + ii) * g.dh, 1);
          }
          tok_tab[buf][et] = e;
        }
        // (a warp can be at most one tile ahead of the slowest: it passes this barrier only after every warp has left
        // the tile before, so the table of the tile before that is free to be overwritten)
        asm volatile("bar.sync %0, %1;" ::"n"(BAR_PEPI), "n"(NPEPI) : "memory");
      } else {
        const int f = nt * 64 + cl;
        if (g.scale_g) s_lo = g.scale_g[f];
        if (g.scale_u) s_hi = g.scale_u[f];
      }
      // q | k tiles: (cos, sin) of this lane's rotary pair at its 8 tokens of a 16-column chunk, requested one chunk ahead
      // (the first chunk's before the accumulator is complete)
      float2 cs_next[8];
      const bool rot_tile = QKV && nt * 128 < (g.Hq + g.Hkv) * g.dh && g.rope != nullptr;
      const int pidx_tile = QKV ? ((((nt * 128) % g.dh) >> 7) * 64 + cl) : 0;   // rotary pair: channels pidx, pidx + dh / 2
      const float2* const rope_p = g.rope + pidx_tile;
      auto fetch_cs = [&](int c0) {
#pragma unroll
        for (int j = 0; j < 8; ++j) cs_next[j] = __ldg(rope_p + tok_tab[buf][c0 + 8 * hi + j].x);
      };
      if constexpr (QKV) {
        if (rot_tile) fetch_cs(hf * 64);
      }
      // (after a wait that did not even end within the drain bound the warp keeps walking its tiles, without waiting
      // and without stores: the other warps meet it at the table barrier of every tile)
      int r = 0;
      if (!dead) {
        if (lane == 0) r = mbar_wait_drain(smem_u32(&bar_tfull[buf]), ((uint32_t)i >> 1) & 1u, wc);
        r = __shfl_sync(0xffffffffu, r, 0);
        if (r < 0) dead = true;
      }
      const bool ok = !dead && r > 0 && !*reinterpret_cast<volatile int*>(&abort_flag);
      tc_fence_after();
      if (i == 0 && ew == 0 && lane == 0) trace_stamp(trc, 5);
      // q | k | v: what this tile is
      const int Nq = g.Hq * g.dh, Nk = g.Hkv * g.dh, n0 = nt * 128;
      const bool rot = QKV && n0 < Nq + Nk;     // q or k tile: 64 first-half channels and their rotary partners
      const bool isq = n0 < Nq;
      const int nn = isq ? n0 : (rot ? n0 - Nq : n0 - Nq - Nk);
      const int head = QKV ? nn / g.dh : 0;
      const int coff = nn - head * g.dh;        // v: first of the tile's 128 channels; q / k: 128 x (64-channel slice)
      const int half = g.dh >> 1;
      if (QKV && isq) {   // q leaves scaled by 1 / sqrt(dh): folded into the row scales (the rotation is linear)
        const float osc = rsqrtf((float)g.dh);
        s_lo *= osc, s_hi *= osc;
      }
      // gate / up: the tile's k-chunk of the output image; q / k: this lane's rotary pair in the tile's head; v: this
      // lane's channel in the tile's head (the token's row offset comes from the table)
      __nv_bfloat16* const obase =
          !QKV ? g.out_tiled + (size_t)nt * g.rows_pad * 64 + (size_t)(cl & 7)
               : (rot ? (isq ? g.qr : g.kr) + (size_t)head * g.S * g.dh + pidx_tile
                      : g.vr + (size_t)head * g.S * g.dh + coff + 64 * hi + cl);
#pragma unroll 1
      for (int c0 = hf * 64; c0 < hf * 64 + 64; c0 += 16) {
        float v[16];
        tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * GU_NT + c0), v);
        if (c0 == hf * 64 + 48) {
          // this warp has read its part of the accumulator: the MMAs of the tile after next may overwrite it
          tc_fence_before();
          if (lane == 0) mbar_arrive_local(smem_u32(&bar_tempty[buf]));
        }
        if (QKV && !rot) {
          // v tile: lane = channel 64 hi + cl of the tile (the rows are interleaved like those of the q / k tiles), 16
          // token columns each
          const float sc = hi ? s_hi : s_lo;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int tl = c0 + j, tok = tok_base + tl;
            float x = v[j] * sc;
            if constexpr (F8) x *= tok < g.M ? __ldg(g.xscale + tok) : 0.f;
            const int4 e = tok_tab[buf][tl];
            if (ok && e.w) obase[e.z] = __float2bfloat16_rn(x);
          }
          continue;
        }
        // gate (first-half) lanes take the tile's token columns c0 .. c0 + 7, up (partner) lanes c0 + 8 .. c0 + 15: each
        // sends the other half to its partner lane (lane ^ 16)
        const int tl0 = c0 + 8 * hi;
        float2 cs_cur[8];
        if constexpr (QKV) {
#pragma unroll
          for (int j = 0; j < 8; ++j) cs_cur[j] = cs_next[j];
          if (rot_tile && c0 + 16 < hf * 64 + 64) fetch_cs(c0 + 16);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float mine = hi ? v[8 + j] : v[j];
          const float send = hi ? v[j] : v[8 + j];
          const float recv = __shfl_xor_sync(0xffffffffu, send, 16);
          float lo = (hi ? recv : mine) * s_lo, up = (hi ? mine : recv) * s_hi;
          const int tok = tok_base + tl0 + j;
          if constexpr (F8) {
            const float xs = tok < g.M ? __ldg(g.xscale + tok) : 0.f;
            lo *= xs, up *= xs;
          }
          if constexpr (QKV) {
            const int4 e = tok_tab[buf][tl0 + j];
            if (g.rope) {
              const float2 cs = cs_cur[j];
              const float l2 = lo * cs.x - up * cs.y, u2 = up * cs.x + lo * cs.y;
              lo = l2, up = u2;
            }
            __nv_bfloat16* dst = obase + (isq ? e.y : e.z);
            if (ok && e.w) dst[0] = __float2bfloat16_rn(lo), dst[half] = __float2bfloat16_rn(up);
          } else {
            const float val = gelu_fast(lo, g.gelu_exact) * up;
            if (ok && tok < g.M) obase[(size_t)tok * 64 + (((cl >> 3) ^ (tok & 7)) << 3)] = __float2bfloat16_rn(val);
          }
        }
      }
    }
    tc_fence_before();
    if (ew == 0 && lane == 0 && trc) {
      unsigned long long t;
      unsigned sm;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
      asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
      trc[6] = t, trc[7] = sm, trc[9] = (unsigned long long)n_my;
    }
  }

  __syncthreads();
  // (every copy has landed by now, also after a give-up: the MMA warp waited for every stage it was sent)
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
    if (lane == 0 && trc) {
      unsigned long long t;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
      trc[8] = t;
    }
  }
}

}  // namespace

bool persist_gemm_supported(int M, int N, int K, int rows_pad, bool fp8) {
  const int kb = fp8 ? 128 : 64;
  return N % 128 == 0 && K % kb == 0 && K >= kb && rows_pad % GU_NT == 0 && (M + GU_NT - 1) / GU_NT * GU_NT <= rows_pad;
}

cudaError_t persist_gemm_setup() {
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k_gemm_persist<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GU_SMEM))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_persist<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GU_SMEM))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_persist<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GU_SMEM))) return e;
  return cudaFuncSetAttribute(k_gemm_persist<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GU_SMEM);
}

int persist_gemm_ctas(const PersistGemm& g, int n_sm) {
  const int n_tiles = (g.N >> 7) * ((g.M + GU_NT - 1) / GU_NT);
  return n_tiles < n_sm ? n_tiles : n_sm;
}

cudaError_t launch_persist_gemm(int* status, const PersistGemm& g, int n_sm, cudaStream_t st) {
  if (!persist_gemm_supported(g.M, g.N, g.K, g.rows_pad, g.fp8 != 0)) return cudaErrorInvalidValue;
  if (g.fp8 && !g.xscale) return cudaErrorInvalidValue;
  if (g.qkv && (!g.rq || g.S > 64 || (g.dh != 128 && g.dh != 256) || g.N != (g.Hq + 2 * g.Hkv) * g.dh)) return cudaErrorInvalidValue;
  const dim3 grid(persist_gemm_ctas(g, n_sm));
  if (g.fp8)
    return g.qkv ? launch_pdl(k_gemm_persist<true, true>, grid, dim3(800), GU_SMEM, st, status, g)
                 : launch_pdl(k_gemm_persist<true, false>, grid, dim3(800), GU_SMEM, st, status, g);
  return g.qkv ? launch_pdl(k_gemm_persist<false, true>, grid, dim3(800), GU_SMEM, st, status, g)
               : launch_pdl(k_gemm_persist<false, false>, grid, dim3(800), GU_SMEM, st, status, g);
}

}  // namespace phyai
