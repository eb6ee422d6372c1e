// bf16 tensor-core GEMM for sm_100a: bulk-copy (TMA engine) staged operands, tcgen05.mma with the
// fp32 accumulator in tensor memory, fused epilogues.
//
// Orientation ("weights on the M axis"): the MMA's 128-row M dimension holds 128 output channels
// of the weight matrix, the N dimension holds NT tokens.  A batch-1 request has only ~51 tokens,
// which would waste a 128-row M tile; as N they cost a 64-wide tile.  Large batches use NT = 128 or
// 256 with the same kernel.  Per output channel (TMEM lane = one epilogue thread) the dequant scale,
// bias and residual gate are per-thread scalars.
//
// Operands: both K-major with the 128-byte swizzle.
//   A: weights pre-packed at create time into [N/128][K/64] blocks of 128 rows x 128 bytes.
//   B: activations kept in the tiled bf16 layout, so an NT x 64 tile is one contiguous block.
// Every load is therefore a 1-D bulk copy (16-byte aligned, size a multiple of 16): no tensor map.
//
// A CTA computes NA (1 or 2) 128-channel tiles against one NT-token tile (NT = 64, 128, 192 or 256): with NA = 2
// and NT = 256 a k-step moves 64 KB for 8 MMAs of 128 clocks, i.e. 64 bytes per clock.  One SM alone ingests that
// (~126 GB/s measured); with all SMs streaming the main loop was measured at ~1180 clocks per k-step (55 bytes per
// clock per SM, 87 % of the tensor rate).  A single 128 x 256 tile would need 96 bytes per clock.  What a 256 x 256
// tile loses is its epilogue and set-up: they cannot overlap a next tile because the accumulators fill the tensor
// memory (see gemm_persist.cu for the projections with more tiles than SMs).
//
// Warp roles (800 threads): warps 0..7 = copy producers (the copies of all stages are dealt round
// robin to the eight warps: one warp's bulk copies complete one at a time, about 0.5 us each whatever
// their size, so many issuing warps are needed to keep the SM's L2 port busy), warp 8 = TMEM owner +
// MMA issuer (whole warp in the loop, one elected lane issues), warps 9..24 = epilogue (TMEM lane
// quarter = warp % 4, token-column quarter = (warp - 9) / 4).  The epilogue of a 256 x 256 tile is not
// overlapped with a next tile (TMEM is full), so it gets 16 warps and batches its global loads.
// Epilogues: plain store, gated residual (read-modify-write; split-K: 16-byte vector reductions, or slabs that the
// next kernel sums in a fixed order), GeGLU (paired gate / up tiles, or interleaved 64 + 64 tiles), bias + row remap,
// and the rotary epilogue of the fused QKV projection (rotated, scaled bf16 q / k / v in the attention layout).
// The kernel is launched with programmatic stream serialization: barriers, TMEM and the weight halves of the first
// STAGES stages are set up before griddepcontrol.wait, i.e. while the kernel producing the activations still runs.
// Every wait is bounded: on expiry of the caller's limit the CTA raises the status word and skips its MMAs and
// stores, but keeps the copy / commit pipeline running under a generous limit of its own, so that every copy
// into its shared memory has landed before it exits (TMEM is always released).
#include "kernels.h"
#include "ptx.cuh"
#include "tc.cuh"

namespace phyai {
namespace {

constexpr int A_BYTES = 128 * 128;  // one weight block: 128 out channels x 64 k (bf16)
constexpr int NPROD = 8;
constexpr int NEPI = 512;           // epilogue threads (16 warps)
constexpr int BAR_EPI = 1;

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync %0, %1;" ::"n"(BAR_EPI), "n"(NEPI) : "memory"); }

// F8: e4m3 operands (kind::f8f6f4) and per-token activation scales, a kernel of its own so that the bf16 kernel carries
// none of it.
template <int NT, int NA, int STAGES, bool F8 = false>
__global__ void __launch_bounds__(800, 1) k_gemm_tc(int* status, const TcGemm g) {
  constexpr int B_BYTES = NT * 128;
  constexpr int NB = NT > 128 ? NT / 128 : 1;          // the activation tile is copied in pieces of <= 16 KB
  constexpr int B_PIECE = B_BYTES / NB;
  constexpr int NCOPY = NA + NB;
  constexpr int STAGE_BYTES = A_BYTES * NA + B_BYTES;
  // Single 64-token tile: two warps issue MMAs, one the even k-steps, one the odd ones, each into an accumulator of
  // its own (the epilogue adds the two).  The issue sequence of a k-step (four N = 64 MMAs of ~55 clocks each)
  // takes one thread ~350 clocks plus the wait for the next stage, so a single issuer, not the tensor pipe, set
  // the pace of these launches.
  constexpr bool DUAL = NT == 64 && NA == 1;
  constexpr int COLS = NA * NT * (DUAL ? 2 : 1);
  constexpr int ALLOC_COLS = COLS <= 32 ? 32 : COLS <= 64 ? 64 : COLS <= 128 ? 128 : COLS <= 256 ? 256 : 512;   // power of two
  // A producer warp's consecutive copies are NPROD / NCOPY k-steps apart; its parity wait on "stage free" is only
  // meaningful while that step does not exceed the ring depth.
  // Copy issuers: the 8 producer warps, plus (single 64-token tile) the first epilogue warps, which are idle during
  // the main loop.  One warp's bulk copies complete one at a time (measured), so the number of copies in flight is
  // the number of issuing warps: with 8 issuers a 16-step main loop of 32 copies took 4.9 us whatever was prefetched.
  constexpr int NISSUE = (NT == 64 && NA == 1) ? (2 * STAGES < 24 ? 2 * STAGES : 24) : NPROD;
  static_assert((NISSUE + NCOPY - 1) / NCOPY <= STAGES, "producer stride exceeds the stage ring");
  // instruction descriptor: D fp32 (bit 4), A bf16 (bit 7), B bf16 (bit 10), both K-major,
  // N >> 3 at bit 17, M >> 4 at bit 24.
  constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NT >> 3) << 17) | ((128u >> 4) << 24);
  // e4m3 x e4m3 (kind::f8f6f4): format fields 0, fp32 accumulation
  constexpr uint32_t IDESC_F8 = (1u << 4) | ((uint32_t)(NT >> 3) << 17) | ((128u >> 4) << 24);

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[STAGES];
  __shared__ __align__(8) uint64_t bar_empty[STAGES];
  __shared__ __align__(8) uint64_t bar_accum;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int skip_flag;
  __shared__ int epi_ok;
  __shared__ int2 tok_tab[NT];   // TC_QKV_ROT: per token of the tile (position, request * 64 + suffix row)

  // The warp index and the tensor-memory base are broadcast from lane 0: the compiler then knows that they are the
  // same in every lane, keeps the role branches and the MMA operands (descriptors, addresses) in the uniform
  // datapath, and the issue sequence of one k-step shrinks (measured in a stand-alone model of this main loop:
  // 530 -> 410 clocks per k-step of four N = 64 MMAs).
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const int nt_idx = blockIdx.x, tt = blockIdx.y;
  const bool geglu = g.epi == TC_GEGLU;
  const int KC = F8 ? g.K >> 7 : g.K >> 6;   // k-chunks of 128 bytes per operand row
  const int kc_begin = (int)(((long long)KC * blockIdx.z) / gridDim.z);
  const int kc_end = (int)(((long long)KC * (blockIdx.z + 1)) / gridDim.z);
  const int nk = kc_end - kc_begin;

  // Programmatic dependent launch: this grid may start while the kernel before it is still running.  Everything up
  // to pdl_wait() touches only shared / tensor memory and the weights (constants): barriers, TMEM, and the weight
  // halves of the first STAGES stages are in flight before the activations this GEMM depends on exist.
  pdl_launch_dependents();
  unsigned long long* const trc =
      g.trace ? g.trace + (size_t)((blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) * 16 : nullptr;
  if (threadIdx.x == 0) trace_stamp(trc, 0);
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* tiles_ptr = smem_raw + (tiles - smem_u32(smem_raw));
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bar_full[s]), NCOPY);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    mbar_init(smem_u32(&bar_accum), DUAL ? 2 : 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    tmem_alloc(smem_u32(&tmem_slot), ALLOC_COLS);
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  if (threadIdx.x == 0) trace_stamp(trc, 1);
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, *reinterpret_cast<volatile uint32_t*>(&tmem_slot), 0);
  const WaitCtx wc{status, &abort_flag, g.wait_limit};

  // weight tile of accumulator a: GeGLU pairs the gate and up tiles of the same channels, otherwise
  // a CTA owns NA consecutive tiles
  auto wtile = [&](int a) -> const uint8_t* {
    const __nv_bfloat16* base = (geglu && a == 1) ? g.W2 : g.W;
    const int tile = geglu ? nt_idx : nt_idx * NA + a;
    return reinterpret_cast<const uint8_t*>(base) + ((size_t)tile * KC + kc_begin) * A_BYTES;
  };
  const int n_early = nk < STAGES ? (nk > 0 ? nk : 0) : STAGES;   // stages whose weight copies are issued before the wait
  // copy issuers: producer warps 0..7, then the epilogue warps that are idle during the main loop (with two MMA
  // warps the first epilogue warp is not)
  const int issuer = warp < NPROD ? warp : warp - (DUAL ? 2 : 1);
  const bool issues = lane == 0 && warp != 8 && !(DUAL && warp == 9) && issuer < NISSUE;
  if (issues) {
    for (int id = issuer; id < n_early * NCOPY; id += NISSUE) {
      const int i = id / NCOPY, c = id % NCOPY;
      if (c >= NA) continue;
      const uint32_t full = smem_u32(&bar_full[i]);
      mbar_expect_tx(full, A_BYTES);
      bulk_g2s(tiles + (uint32_t)i * STAGE_BYTES + c * A_BYTES, wtile(c) + (size_t)i * A_BYTES, A_BYTES, full);
    }
  }
  pdl_wait();
  if (threadIdx.x == 0) trace_stamp(trc, 2);
  // The activation copies of the prefetched stages go out before the status word is known (their addresses do not
  // depend on the request, and the skip path below waits for them): the status read, a round trip to the L2, then
  // overlaps their latency.  It is made by the MMA warp, which issues no copies.
  const uint8_t* xsrc = reinterpret_cast<const uint8_t*>(g.X) + ((size_t)kc_begin * g.rows_pad + (size_t)tt * NT) * 128;
  auto issue_x = [&](int i, int pc, uint32_t s_idx) {
    const uint32_t full = smem_u32(&bar_full[s_idx]);
    mbar_expect_tx(full, B_PIECE);
    bulk_g2s(tiles + s_idx * STAGE_BYTES + NA * A_BYTES + pc * B_PIECE, xsrc + (size_t)i * g.rows_pad * 128 + (size_t)pc * B_PIECE,
             B_PIECE, full);
  };
  if (issues) {
    if constexpr (NT == 64 && NA == 1) {
      // Concurrent copies share the SM's ingest rate, so with one issuer per stage all activation tiles would land
      // together, late; XW issuers taking the stages round robin (a warp's copies complete in order) bring the
      // first stages in first.
      constexpr int XW = 3;   // 1 / 2 / 3 / 5 / 9 issuers measured 7.26 / 7.23 / 7.19 / 7.18 / 7.20 ms per batch-1 chunk
      if (issuer < XW)
        for (int i = issuer; i < n_early; i += XW) issue_x(i, 0, (uint32_t)i);
    } else {
      for (int id = issuer; id < n_early * NCOPY; id += NISSUE)
        if (id % NCOPY >= NA) issue_x(id / NCOPY, id % NCOPY - NA, (uint32_t)(id / NCOPY));
    }
  }
  if (threadIdx.x == NPROD * 32) skip_flag = status_set(status) || nk <= 0;
  __syncthreads();
  if (skip_flag) {
    // every copy issued so far must land before this CTA's shared memory is released (a wait on this CTA's own
    // copies: bounded by the drain limit, not by the caller's)
    if (threadIdx.x == 0)
      for (int i = 0; i < n_early; ++i) mbar_wait_drain(smem_u32(&bar_full[i]), 0u, wc);
    __syncthreads();
    if (warp == 8) {
      tc_fence_after();
      tmem_dealloc(tmem_base, ALLOC_COLS);
    }
    return;
  }

  // ---------------- copy issuers: copy number id = k-step * NCOPY + piece goes to issuer id % NISSUE --------------
  if (issues) {
    for (int id = issuer + (n_early * NCOPY - issuer + NISSUE - 1) / NISSUE * NISSUE; id < nk * NCOPY; id += NISSUE) {
      const int i = id / NCOPY, c = id % NCOPY;
      const int s = i % STAGES;
      const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
      // (after a give-up the pipeline keeps running -- copies, commits and barriers as usual, MMAs and stores
      // skipped -- so that nothing is in flight when the CTA exits)
      if (mbar_wait_drain(smem_u32(&bar_empty[s]), ph ^ 1u, wc) < 0) break;
      if (c < NA) {
        const uint32_t full = smem_u32(&bar_full[s]);
        mbar_expect_tx(full, A_BYTES);
        bulk_g2s(tiles + (uint32_t)s * STAGE_BYTES + c * A_BYTES, wtile(c) + (size_t)i * A_BYTES, A_BYTES, full);
      } else {
        issue_x(i, c - NA, (uint32_t)s);
      }
    }
  }
  __syncwarp();
  if (warp == 8 || (DUAL && warp == 9)) {
    // ---------------- MMA issuer(s) (whole warp in the loop, one elected lane issues) ---------------------
    const int first = DUAL ? warp - 8 : 0, step = DUAL ? 2 : 1;
    const uint32_t tacc = tmem_base + (DUAL ? (uint32_t)(warp - 8) * NT : 0u);
    for (int i = first; i < nk; i += step) {
      const int s = i % STAGES;
      const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
      const bool ok = mbar_wait_drain(smem_u32(&bar_full[s]), ph, wc) > 0;
      if (i == 0 && lane == 0) trace_stamp(trc, 3);
      // (no tcgen05 fence here: the operands were written by the bulk-copy engine and made visible by the mbarrier;
      // tcgen05.fence::after_thread_sync orders tensor-memory accesses, and it was measured to hold the next MMAs
      // back until the previous stage's MMAs had drained)
      const uint32_t a0 = tiles + (uint32_t)s * STAGE_BYTES;
      const uint64_t da = make_desc(a0);
      const uint64_t da2 = make_desc(a0 + A_BYTES);
      const uint64_t db = make_desc(a0 + A_BYTES * NA);
      // control flow and descriptors stay warp-uniform; only the tcgen05 instructions themselves are predicated on
      // the elected lane
      if (__all_sync(0xffffffffu, ok)) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {  // 4 x (K = 16) per 64-wide chunk: +32 bytes = +2 descriptor units
          const uint32_t acc = (i > first || k > 0) ? 1u : 0u;   // the warp's first MMA initialises its accumulator
          if constexpr (F8) {
            if (elect_one()) umma_f8(tacc, da + 2 * k, db + 2 * k, IDESC_F8, acc);
            if (NA == 2) {
              if (elect_one()) umma_f8(tacc + NT, da2 + 2 * k, db + 2 * k, IDESC_F8, acc);
            }
          } else {
            if (elect_one()) umma_bf16(tacc, da + 2 * k, db + 2 * k, IDESC, acc);
            if (NA == 2) {
              if (elect_one()) umma_bf16(tacc + NT, da2 + 2 * k, db + 2 * k, IDESC, acc);
            }
          }
        }
      }
      // frees the stage when the MMAs above have read it -- only if a later k-step will reuse the stage (a commit
      // that nobody waits for still costs the issuing thread time)
      if (i + STAGES < nk && elect_one()) umma_commit(smem_u32(&bar_empty[s]));
      __syncwarp();
    }
    if (elect_one()) umma_commit(smem_u32(&bar_accum));
    __syncwarp();
    if (warp == 8 && lane == 0) trace_stamp(trc, 4);
  }
  if (warp <= 8) {
    // (producer warps and the first MMA warp have nothing else to do)
  } else {
    // ---------------- epilogue: TMEM -> registers -> global --------------------------------------
    const int ew = warp - 9;                      // 0..15
    const int q = warp & 3, hf = ew >> 2;         // TMEM lane quarter, token-column quarter
    const int et = ew * 32 + lane;                // 0..511
    const int ch = q * 32 + lane;                 // row of the 128-row tile
    const int tok_base = tt * NT;
    // 16 accumulator columns of this thread's TMEM lane (two MMA warps: the sum of their accumulators)
    // W8A8: activation scale of every token of the tile.  The table sits at the end of the operand stages, which are
    // free once the accumulator is complete; the values are fetched into registers while the main loop still runs.
    float* xs_tab = reinterpret_cast<float*>(tiles_ptr + (size_t)STAGES * STAGE_BYTES) - NT;
    // (W8A8: times the activation scale of each column's token)
    auto ld_acc = [&](uint32_t col, float* v) {
      tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + col, v);
      if (DUAL && nk > 1) {
        float w[16];
        tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)NT + col, w);
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] += w[j];
      }
      if constexpr (F8) {
        const float* xs = xs_tab + (col % (uint32_t)NT);
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] *= xs[j];
      }
    };
    float xs_reg = 0.f;
    if (F8 && et < NT && tok_base + et < g.M) xs_reg = g.xscale[tok_base + et];
    if (g.epi == TC_QKV_ROT) {
      // while the main loop runs: where each token of the tile sits (request, suffix row, rotary position)
      for (int idx = et; idx < NT; idx += NEPI) {
        const int tok = tok_base + idx;
        int2 e = make_int2(0, 0);
        if (tok < g.M) {
          const int b = tok / g.S, i = tok - b * g.S;
          const int* cu = g.rq->cu_lens;
          e = make_int2(cu[b + 1] - cu[b] + i, b * 64 + i);
        }
        tok_tab[idx] = e;
      }
    }
    // per-channel constants of the plain epilogues (weight scale, residual gate, bias) are fetched while the main
    // loop runs, not after the accumulator is ready
    float e_sc[NA], e_gt[NA], e_bs[NA], e_il = 1.0f;
    if (!geglu && g.epi != TC_QKV_ROT && g.epi != TC_GEGLU_IL) {
#pragma unroll
      for (int a = 0; a < NA; ++a) {
        const int n = (nt_idx * NA + a) * 128 + ch;
        e_sc[a] = g.scale ? g.scale[n] : 1.0f;
        e_gt[a] = (g.epi == TC_RESID && g.gate) ? g.gate[n] : 1.0f;
        e_bs[a] = (g.epi == TC_BIAS_ROWMAP && g.bias) ? g.bias[n] : 0.0f;
      }
    } else {
#pragma unroll
      for (int a = 0; a < NA; ++a) e_sc[a] = e_gt[a] = 1.0f, e_bs[a] = 0.0f;
      if (g.epi == TC_GEGLU_IL) {
        const int f = nt_idx * 64 + (ch & 63);
        const float* sp = q >= 2 ? g.scale2 : g.scale;
        if (sp) e_il = sp[f];
      }
    }
    // rotary epilogue: the weight scale and the table rows of this thread's first item of accumulator 0 are on
    // their way before the accumulator is ready (the later ones are requested one item ahead)
    float4 cs_pre[4];
    int2 e_pre = make_int2(0, 0);
    float sc_pre = 1.0f;
    bool pre = false;
    if (g.epi == TC_QKV_ROT) {
      epi_sync();                                   // tok_tab complete
      const int n0 = nt_idx * NA * 128;
      if (g.scale) sc_pre = g.scale[n0 + ch];
      const int rows = min(NT, g.M - tok_base);
      const int Nq = g.Hq * g.dh, Nk = g.Hkv * g.dh;
      if (n0 < Nq + Nk && et < rows * 8) {
        const int nn = n0 < Nq ? n0 : n0 - Nq;
        const int t = (nn % g.dh) >> 7;
        e_pre = tok_tab[et >> 3];
        pre = true;
        if (g.rope) {
          const float4* cs = reinterpret_cast<const float4*>(g.rope + (size_t)e_pre.x * (g.dh >> 1) + t * 64 + (et & 7) * 8);
#pragma unroll
          for (int u = 0; u < 4; ++u) cs_pre[u] = __ldg(cs + u);
        }
      }
    }
    // one epilogue warp polls the accumulator barrier; the other fifteen wait for it at the named barrier (in
    // hardware), so that the main loop's shared-memory port is not shared with 512 polling threads
    if (ew == 0) {
      const bool okw = mbar_wait_drain(smem_u32(&bar_accum), 0, wc) > 0;
      if (lane == 0) epi_ok = okw ? 1 : 0;
    }
    epi_sync();
    const bool ok = *reinterpret_cast<volatile int*>(&epi_ok) != 0;
    tc_fence_after();
    if (et == 0) trace_stamp(trc, 5);
    if constexpr (F8) {
      if (et < NT) xs_tab[et] = xs_reg;
      epi_sync();
    }
    constexpr int HALF = NT / 4;   // token columns per epilogue warp
    const int c_begin = hf * HALF;
    const bool resid_red = g.epi == TC_RESID && gridDim.z > 1;   // split-K: vector reductions, see below
    if (ok && !geglu && g.epi != TC_QKV_ROT && g.epi != TC_GEGLU_IL && !resid_red) {
#pragma unroll
      for (int a = 0; a < NA; ++a) {
        const int n = (nt_idx * NA + a) * 128 + ch;   // packed output channel
        const float sc = e_sc[a];
        const int n_out = (g.perm_dh && n < g.perm_end) ? qkv_packed_to_channel(n, g.perm_dh) : n;
        const float gt = e_gt[a];
        const float bs = e_bs[a];
#pragma unroll 1
        for (int c0 = c_begin; c0 < c_begin + HALF; c0 += 16) {
          if (tok_base + c0 >= g.M) break;  // warp-uniform
          float v[16];
          ld_acc((uint32_t)(a * NT + c0), v);
          if (g.epi == TC_RESID && gridDim.z == 1) {
            // single owner per element: plain read-modify-write, with the 16 loads issued before any is used
            float old[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int tok = tok_base + c0 + j;
              old[j] = tok < g.M ? g.out_f32[(size_t)tok * g.ldo + n] : 0.f;
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int tok = tok_base + c0 + j;
              if (tok < g.M) g.out_f32[(size_t)tok * g.ldo + n] = old[j] + gt * (v[j] * sc);
            }
            continue;
          }
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int tok = tok_base + c0 + j;
            if (tok < g.M) {
              const float val = v[j] * sc;
              if (g.epi == TC_STORE) {
                g.out_f32[(size_t)tok * g.ldo + n_out] = val;
              } else if (g.epi == TC_RESID) {
                atomicAdd(&g.out_f32[(size_t)tok * g.ldo + n], gt * val);
              } else {
                const int orow = (tok / g.rows_in) * g.rows_out + g.row_off + tok % g.rows_in;
                g.out_f32[(size_t)orow * g.ldo + n] = val + bs;
              }
            }
          }
        }
      }
    }
    if (g.epi == TC_GEGLU_IL) {
      // One 128-row tile = 64 gate channels (rows 0..63) and the matching 64 up channels (rows 64..127): twice as
      // many CTAs stream the gate / up weights as with separate 128-row gate and up tiles, which is what matters
      // when there is a single token tile.  The up half goes through shared memory to the gate half, which writes
      // the bf16 result as the swizzled image of k-chunk `tile` of the down projection's input.
      float* stage = reinterpret_cast<float*>(tiles_ptr);                                  // [NT][64] up values
      __nv_bfloat16* img = reinterpret_cast<__nv_bfloat16*>(stage + (size_t)NT * 64);      // [NT][64] bf16, swizzled
      const int c64 = ch & 63;
      float gel[HALF / 16][16];   // gate half: gelu(gate), computed while the up half is on its way through shared memory
      if (ok) {
#pragma unroll
        for (int u = 0; u < HALF / 16; ++u) {
          const int c0 = c_begin + u * 16;
          if (tok_base + c0 >= g.M) break;
          float v[16];
          ld_acc((uint32_t)c0, v);
          if (q >= 2) {
#pragma unroll
            for (int j = 0; j < 16; ++j) stage[(size_t)(c0 + j) * 64 + c64] = v[j] * e_il;
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) gel[u][j] = gelu_fast(v[j] * e_il, g.gelu_exact);
          }
        }
      }
      epi_sync();
      if (ok && q < 2) {
#pragma unroll
        for (int u = 0; u < HALF / 16; ++u) {
          const int c0 = c_begin + u * 16;
          if (tok_base + c0 >= g.M) break;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int t = c0 + j;
            const float m = gel[u][j] * stage[(size_t)t * 64 + c64];
            img[(size_t)t * 64 + (((c64 >> 3) ^ (t & 7)) << 3) + (c64 & 7)] = __float2bfloat16_rn(m);
          }
        }
      }
      epi_sync();
      if (ok) {
        const int rows = min(NT, g.M - tok_base);
        uint4* dst = reinterpret_cast<uint4*>(g.out_tiled + ((size_t)nt_idx * g.rows_pad + tok_base) * 64);
        const uint4* src = reinterpret_cast<const uint4*>(img);
#pragma unroll 1
        for (int idx = et; idx < rows * 8; idx += NEPI) dst[idx] = src[idx];
      }
    }
    if (resid_red) {
      // Split-K residual: every k-range adds its partial tile to h.  The tile is transposed through shared memory
      // (fp32 [token][128 + 4]) so that one thread adds 4 consecutive channels of one token with a single
      // 16-byte reduction: a quarter of the reduction operations of per-element atomics, in whole 128-byte lines.
      constexpr int PITCH = 132;
      float* stage = reinterpret_cast<float*>(tiles_ptr);
      const int rows = min(NT, g.M - tok_base);
#pragma unroll 1
      for (int a = 0; a < NA; ++a) {
        const int n0 = (nt_idx * NA + a) * 128;
        if (ok) {
          const float sc = e_sc[a] * e_gt[a];
#pragma unroll 1
          for (int c0 = c_begin; c0 < c_begin + HALF; c0 += 16) {
            if (tok_base + c0 >= g.M) break;          // warp-uniform
            float v[16];
            ld_acc((uint32_t)(a * NT + c0), v);
#pragma unroll
            for (int j = 0; j < 16; ++j) stage[(size_t)(c0 + j) * PITCH + ch] = v[j] * sc;
          }
        }
        epi_sync();
        if (ok) {
#pragma unroll 1
          for (int it = et; it < rows * 32; it += NEPI) {
            const int tl = it >> 5, j0 = (it & 31) * 4;
            const float4 x = *reinterpret_cast<const float4*>(stage + (size_t)tl * PITCH + j0);
            if (g.slab) {   // deterministic variant: plain stores of this k-range's partial
              *reinterpret_cast<float4*>(g.slab + ((size_t)blockIdx.z * g.M + tok_base + tl) * g.ldo + n0 + j0) = x;
              continue;
            }
            float* dst = g.out_f32 + (size_t)(tok_base + tl) * g.ldo + n0 + j0;
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(x.x), "f"(x.y), "f"(x.z), "f"(x.w)
                         : "memory");
          }
        }
        epi_sync();
      }
    }
    if (g.epi == TC_QKV_ROT) {
      // Each accumulator is one 128-row tile of the packed q|k|v matrix: 64 channels of the first half of a head
      // followed by their rotary partners (or 128 v channels).  The tile is transposed through shared memory
      // (the stages are free: every MMA has completed) as fp32 [token][128 + 4]; then one thread takes 8
      // channels and their partners of one token, rotates, and writes two 16-byte bf16 runs.
      constexpr int PITCH = 132;
      float* stage = reinterpret_cast<float*>(tiles_ptr);
      const int half = g.dh >> 1;
      const int rows = min(NT, g.M - tok_base);
      const int Nq = g.Hq * g.dh, Nk = g.Hkv * g.dh;
      const float qscale = rsqrtf((float)g.dh);
#pragma unroll 1
      for (int a = 0; a < NA; ++a) {
        const int n0 = (nt_idx * NA + a) * 128;       // first packed row of this accumulator
        if (ok) {
          const float sc = a == 0 ? sc_pre : (g.scale ? g.scale[n0 + ch] : 1.0f);
#pragma unroll 1
          for (int c0 = c_begin; c0 < c_begin + HALF; c0 += 16) {
            if (tok_base + c0 >= g.M) break;          // warp-uniform
            float v[16];
            ld_acc((uint32_t)(a * NT + c0), v);
#pragma unroll
            for (int j = 0; j < 16; ++j) stage[(size_t)(c0 + j) * PITCH + ch] = v[j] * sc;
          }
        }
        epi_sync();
        if (ok) {
          if (n0 < Nq + Nk) {
            const bool isq = n0 < Nq;
            const int nn = isq ? n0 : n0 - Nq;
            const int head = nn / g.dh, t = (nn - head * g.dh) >> 7;   // 64-channel slice of the head's first half
            __nv_bfloat16* base = isq ? g.qr : g.kr;
            const int H = isq ? g.Hq : g.Hkv;
            const float osc = isq ? qscale : 1.0f;
            // the rotary table rows of the next item are requested before this item is processed
            float4 cs_next[4];
            int2 e_next = make_int2(0, 0);
            auto fetch = [&](int it2) {
              e_next = tok_tab[it2 >> 3];
              if (g.rope) {
                const float4* cs = reinterpret_cast<const float4*>(g.rope + (size_t)e_next.x * half + t * 64 + (it2 & 7) * 8);
#pragma unroll
                for (int u = 0; u < 4; ++u) cs_next[u] = __ldg(cs + u);
              }
            };
            if (a == 0 && pre) {
              e_next = e_pre;
#pragma unroll
              for (int u = 0; u < 4; ++u) cs_next[u] = cs_pre[u];
            } else if (et < rows * 8) {
              fetch(et);
            }
#pragma unroll 1
            for (int it = et; it < rows * 8; it += NEPI) {
              const int tl = it >> 3, j0 = (it & 7) * 8;
              const int2 e = e_next;
              float4 csc[4];
#pragma unroll
              for (int u = 0; u < 4; ++u) csc[u] = cs_next[u];
              if (it + NEPI < rows * 8) fetch(it + NEPI);
              const float* sp = stage + (size_t)tl * PITCH + j0;
              float lo[8], hi[8];
              *reinterpret_cast<float4*>(lo) = *reinterpret_cast<const float4*>(sp);
              *reinterpret_cast<float4*>(lo + 4) = *reinterpret_cast<const float4*>(sp + 4);
              *reinterpret_cast<float4*>(hi) = *reinterpret_cast<const float4*>(sp + 64);
              *reinterpret_cast<float4*>(hi + 4) = *reinterpret_cast<const float4*>(sp + 68);
              if (g.rope) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                  const float4 c = csc[u];           // (cos, sin) of channels 2u and 2u + 1
                  const float l0 = lo[2 * u], h0 = hi[2 * u], l1 = lo[2 * u + 1], h1 = hi[2 * u + 1];
                  lo[2 * u] = l0 * c.x - h0 * c.y, hi[2 * u] = h0 * c.x + l0 * c.y;
                  lo[2 * u + 1] = l1 * c.z - h1 * c.w, hi[2 * u + 1] = h1 * c.z + l1 * c.w;
                }
              }
              const int b = e.y >> 6, i = e.y & 63;
              __nv_bfloat16* dst = base + ((size_t)(b * H + head) * g.S + i) * g.dh + t * 64 + j0;
              auto pk = [&](const float* x) {
                __nv_bfloat162 p0 = __floats2bfloat162_rn(x[0] * osc, x[1] * osc), p1 = __floats2bfloat162_rn(x[2] * osc, x[3] * osc);
                __nv_bfloat162 p2 = __floats2bfloat162_rn(x[4] * osc, x[5] * osc), p3 = __floats2bfloat162_rn(x[6] * osc, x[7] * osc);
                return make_uint4(*reinterpret_cast<uint32_t*>(&p0), *reinterpret_cast<uint32_t*>(&p1),
                                  *reinterpret_cast<uint32_t*>(&p2), *reinterpret_cast<uint32_t*>(&p3));
              };
              *reinterpret_cast<uint4*>(dst) = pk(lo);
              *reinterpret_cast<uint4*>(dst + half) = pk(hi);
            }
          } else {
            const int nn = n0 - Nq - Nk;
            const int head = nn / g.dh, coff = nn - head * g.dh;       // 128 consecutive v channels
#pragma unroll 1
            for (int it = et; it < rows * 16; it += NEPI) {
              const int tl = it >> 4, j0 = (it & 15) * 8;
              const int2 e = tok_tab[tl];
              const float* sp = stage + (size_t)tl * PITCH + j0;
              float x[8];
              *reinterpret_cast<float4*>(x) = *reinterpret_cast<const float4*>(sp);
              *reinterpret_cast<float4*>(x + 4) = *reinterpret_cast<const float4*>(sp + 4);
              const int b = e.y >> 6, i = e.y & 63;
              __nv_bfloat162 p0 = __floats2bfloat162_rn(x[0], x[1]), p1 = __floats2bfloat162_rn(x[2], x[3]);
              __nv_bfloat162 p2 = __floats2bfloat162_rn(x[4], x[5]), p3 = __floats2bfloat162_rn(x[6], x[7]);
              *reinterpret_cast<uint4*>(g.vr + ((size_t)(b * g.Hkv + head) * g.S + i) * g.dh + coff + j0) =
                  make_uint4(*reinterpret_cast<uint32_t*>(&p0), *reinterpret_cast<uint32_t*>(&p1),
                             *reinterpret_cast<uint32_t*>(&p2), *reinterpret_cast<uint32_t*>(&p3));
            }
          }
        }
        epi_sync();
      }
    }
    if (geglu) {
      // accumulator 0 = gate, 1 = up of channels nt_idx*128 .. +127.  The bf16 result is built in shared
      // memory as the swizzled image of two k-chunks of the down projection's input (the stages are
      // free: every MMA has completed), then copied out with 16-byte stores.
      __nv_bfloat16* img = reinterpret_cast<__nv_bfloat16*>(tiles_ptr);   // [2][NT][64]
      if (ok) {
        const int n = nt_idx * 128 + ch;
        const float sg = g.scale ? g.scale[n] : 1.0f, su = g.scale2 ? g.scale2[n] : 1.0f;
        const int kc_sel = ch >> 6, c64 = ch & 63;
#pragma unroll 1
        for (int c0 = c_begin; c0 < c_begin + HALF; c0 += 16) {
          if (tok_base + c0 >= g.M) break;
          float vg[16], vu[16];
          tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, vg);
          tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(NT + c0), vu);
          if constexpr (F8) {
#pragma unroll
            for (int j = 0; j < 16; ++j) vg[j] *= xs_tab[c0 + j], vu[j] *= xs_tab[c0 + j];
          }
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int t = c0 + j;   // token within the tile
            const float val = gelu_fast(vg[j] * sg, g.gelu_exact) * (vu[j] * su);
            img[((size_t)kc_sel * NT + t) * 64 + (((c64 >> 3) ^ (t & 7)) << 3) + (c64 & 7)] = __float2bfloat16_rn(val);
          }
        }
      }
      epi_sync();
      if (ok) {
        const int rows = min(NT, g.M - tok_base);
        for (int kc_sel = 0; kc_sel < 2; ++kc_sel) {
          uint4* dst = reinterpret_cast<uint4*>(g.out_tiled + ((size_t)(nt_idx * 2 + kc_sel) * g.rows_pad + tok_base) * 64);
          const uint4* src = reinterpret_cast<const uint4*>(img + (size_t)kc_sel * NT * 64);
#pragma unroll 1
          for (int idx = et; idx < rows * 8; idx += NEPI) dst[idx] = src[idx];
        }
      }
    }
    tc_fence_before();
    if (et == 0 && trc) {
      // (own stores issued; the timer read is tied to this point by the memory clobber)
      unsigned long long t;
      unsigned sm;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
      asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
      trc[6] = t, trc[7] = sm;
    }
  }

  __syncthreads();
  // (every copy has landed by now, also after a give-up: the MMA warps waited for every stage)
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem_base, ALLOC_COLS);
    if (lane == 0 && trc) {
      unsigned long long t;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
      trc[8] = t;
    }
  }
}

template <int NT, int NA, int STAGES>
constexpr size_t smem_bytes() {
  return (size_t)STAGES * (A_BYTES * NA + NT * 128) + 1024;
}

template <int NT, int NA, int STAGES>
cudaError_t launch_one(int* status, const TcGemm& g, cudaStream_t st) {
  dim3 grid(g.N / 128 / (g.epi == TC_GEGLU ? 1 : NA), (g.M + NT - 1) / NT, g.splits > 0 ? g.splits : 1);
  if (g.fp8) {
    if (!g.xscale) return cudaErrorInvalidValue;
    return launch_pdl(k_gemm_tc<NT, NA, STAGES, true>, grid, dim3(800), smem_bytes<NT, NA, STAGES>(), st, status, g);
  }
  return launch_pdl(k_gemm_tc<NT, NA, STAGES, false>, grid, dim3(800), smem_bytes<NT, NA, STAGES>(), st, status, g);
}

template <int NT, int NA, int STAGES>
cudaError_t setup_one() {
  cudaError_t e = cudaFuncSetAttribute(k_gemm_tc<NT, NA, STAGES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem_bytes<NT, NA, STAGES>());
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_gemm_tc<NT, NA, STAGES, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)smem_bytes<NT, NA, STAGES>());
}

}  // namespace

cudaError_t tc_gemm_setup() {
  cudaError_t e;
  if ((e = setup_one<64, 1, 9>()) != cudaSuccess) return e;
  if ((e = setup_one<64, 2, 4>()) != cudaSuccess) return e;
  if ((e = setup_one<128, 1, 5>()) != cudaSuccess) return e;
  if ((e = setup_one<128, 2, 4>()) != cudaSuccess) return e;
  if ((e = setup_one<256, 1, 4>()) != cudaSuccess) return e;
  if ((e = setup_one<256, 2, 3>()) != cudaSuccess) return e;
  if ((e = setup_one<192, 2, 4>()) != cudaSuccess) return e;
  return cudaSuccess;
}

// GeGLU always pairs the gate and up tiles (NA = 2).  Other epilogues take two consecutive channel
// tiles per CTA when the token tile is 256 wide and the channel count allows it (halves the
// activation traffic per MMA), else one.
cudaError_t launch_tc_gemm(int* status, const TcGemm& g, int nt, cudaStream_t st) {
  bool two = g.epi == TC_GEGLU || (nt >= 192 && g.N % 256 == 0 && g.epi != TC_GEGLU_IL);
  // a plain store epilogue cannot split K: when two-tile CTAs would leave more than half of the SMs idle, take one
  // channel tile per CTA instead
  if (g.epi == TC_BIAS_ROWMAP && nt == 256 && (g.N / 256) * ((g.M + 255) / 256) <= 74) two = false;
  if (nt == 64) return two ? launch_one<64, 2, 4>(status, g, st) : launch_one<64, 1, 9>(status, g, st);
  if (nt == 128) return two ? launch_one<128, 2, 4>(status, g, st) : launch_one<128, 1, 5>(status, g, st);
  // 192-token tiles (two channel tiles per CTA only): for token counts where they fill the SMs better
  if (nt == 192 && g.epi != TC_GEGLU && g.N % 256 == 0) return launch_one<192, 2, 4>(status, g, st);
  return two ? launch_one<256, 2, 3>(status, g, st) : launch_one<256, 1, 4>(status, g, st);
}

}  // namespace phyai
