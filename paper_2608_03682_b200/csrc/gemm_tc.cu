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
// Warp roles (288 threads): warps 0..3 = copy producers (stage i is loaded by warp i % 4: one
// warp's bulk copies complete one at a time, about 0.5 us each whatever their size, so several
// issuing warps are needed to keep more than ~30 GB/s per SM in flight), warp 4 = TMEM owner +
// MMA issuer, warps 5..8 = epilogue (TMEM lane quarter = warp % 4).
// Every wait is bounded: on expiry the CTA raises the status word, stops issuing copies, and
// drains to its normal exit (TMEM is always released).
#include "kernels.h"
#include "ptx.cuh"
#include "tc.cuh"

namespace phyai {
namespace {

constexpr int A_BYTES = 128 * 128;  // one weight block: 128 out channels x 64 k (bf16)

template <int NT, bool DUAL, int STAGES>
__global__ void __launch_bounds__(288, 1) k_gemm_tc(int* status, const TcGemm g) {
  constexpr int B_BYTES = NT * 128;
  constexpr int STAGE_BYTES = A_BYTES * (DUAL ? 2 : 1) + B_BYTES;
  constexpr int COLS = DUAL ? 2 * NT : NT;
  // instruction descriptor: D fp32 (bit 4), A bf16 (bit 7), B bf16 (bit 10), both K-major,
  // N >> 3 at bit 17, M >> 4 at bit 24.
  constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NT >> 3) << 17) | ((128u >> 4) << 24);

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[STAGES];
  __shared__ __align__(8) uint64_t bar_empty[STAGES];
  __shared__ __align__(8) uint64_t bar_accum;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int skip_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nt_idx = blockIdx.x, tt = blockIdx.y;
  const int KC = g.K >> 6;
  const int kc_begin = (int)(((long long)KC * blockIdx.z) / gridDim.z);
  const int kc_end = (int)(((long long)KC * (blockIdx.z + 1)) / gridDim.z);
  const int nk = kc_end - kc_begin;

  if (threadIdx.x == 0) {
    skip_flag = status_set(status) || nk <= 0;
    abort_flag = 0;
  }
  __syncthreads();
  if (skip_flag) return;

  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    mbar_init(smem_u32(&bar_accum), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    tmem_alloc(smem_u32(&tmem_slot), COLS);
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  const WaitCtx wc{status, &abort_flag, g.wait_limit};

  constexpr int NPROD = STAGES < 4 ? STAGES : 4;
  if (warp < 4) {
    // ---------------- producers: warp w streams the stages i = w, w + NPROD, ... ---------------------
    if (lane == 0 && warp < NPROD) {
      const uint8_t* wsrc = reinterpret_cast<const uint8_t*>(g.W) + ((size_t)nt_idx * KC + kc_begin) * A_BYTES;
      const uint8_t* wsrc2 =
          DUAL ? reinterpret_cast<const uint8_t*>(g.W2) + ((size_t)nt_idx * KC + kc_begin) * A_BYTES : nullptr;
      const uint8_t* xsrc =
          reinterpret_cast<const uint8_t*>(g.X) + ((size_t)kc_begin * g.rows_pad + (size_t)tt * NT) * 128;
      for (int i = warp; i < nk; i += NPROD) {
        const int s = i % STAGES;
        const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
        if (!mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc)) break;  // stop issuing copies once aborted
        const uint32_t full = smem_u32(&bar_full[s]);
        const uint32_t dst = tiles + (uint32_t)s * STAGE_BYTES;
        mbar_expect_tx(full, STAGE_BYTES);
        bulk_g2s(dst, wsrc + (size_t)i * A_BYTES, A_BYTES, full);
        if (DUAL) bulk_g2s(dst + A_BYTES, wsrc2 + (size_t)i * A_BYTES, A_BYTES, full);
        bulk_g2s(dst + A_BYTES * (DUAL ? 2 : 1), xsrc + (size_t)i * g.rows_pad * 128, B_BYTES, full);
      }
    }
  } else if (warp == 4) {
    // ---------------- MMA issuer (whole warp in the loop, one elected lane issues) ---------------------
    for (int i = 0; i < nk; ++i) {
      const int s = i % STAGES;
      const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
      const bool ok = mbar_wait(smem_u32(&bar_full[s]), ph, wc);
      tc_fence_after();
      const uint32_t a0 = tiles + (uint32_t)s * STAGE_BYTES;
      const uint64_t da = make_desc(a0);
      const uint64_t da2 = make_desc(a0 + A_BYTES);
      const uint64_t db = make_desc(a0 + A_BYTES * (DUAL ? 2 : 1));
      if (elect_one()) {
        if (ok) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {  // 4 x (K = 16) per 64-wide chunk: +32 bytes = +2 descriptor units
            const uint32_t acc = (i > 0 || k > 0) ? 1u : 0u;
            umma_bf16(tmem_base, da + 2 * k, db + 2 * k, IDESC, acc);
            if (DUAL) umma_bf16(tmem_base + NT, da2 + 2 * k, db + 2 * k, IDESC, acc);
          }
        }
        umma_commit(smem_u32(&bar_empty[s]));  // frees the stage when the MMAs above have read it
      }
      __syncwarp();
    }
    if (elect_one()) umma_commit(smem_u32(&bar_accum));
    __syncwarp();
  } else {
    // ---------------- epilogue: TMEM -> registers -> global --------------------------------------
    const int q = warp & 3;
    const int n = nt_idx * 128 + q * 32 + lane;  // this thread's output channel
    const bool ok = mbar_wait(smem_u32(&bar_accum), 0, wc);
    tc_fence_after();
    const float sc = g.scale ? g.scale[n] : 1.0f;
    const int n_out = (g.perm_dh && n < g.perm_end) ? qkv_packed_to_channel(n, g.perm_dh) : n;  // output column
    const int tok_base = tt * NT;
    if (ok) {
      if (!DUAL) {
        const float gt = (g.epi == TC_RESID && g.gate) ? g.gate[n] : 1.0f;
        const float bs = (g.epi == TC_BIAS_ROWMAP && g.bias) ? g.bias[n] : 0.0f;
        for (int c0 = 0; c0 < NT; c0 += 16) {
          if (tok_base + c0 >= g.M) break;  // warp-uniform
          float v[16];
          tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
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
      } else {
        const float sc2 = g.scale2 ? g.scale2[n] : 1.0f;
        for (int c0 = 0; c0 < NT; c0 += 16) {
          if (tok_base + c0 >= g.M) break;
          float vg[16], vu[16];
          tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, vg);
          tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(NT + c0), vu);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int tok = tok_base + c0 + j;
            if (tok < g.M) {
              const float val = gelu_f(vg[j] * sc, g.gelu_exact) * (vu[j] * sc2);
              g.out_tiled[tiled_index(tok, n, g.rows_pad)] = __float2bfloat16_rn(val);
            }
          }
        }
      }
    }
    tc_fence_before();
  }

  __syncthreads();
  if (abort_flag) {
    // give any bulk copy still in flight time to land before shared memory is released
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem_base, COLS);
  }
}

template <int NT, bool DUAL, int STAGES>
constexpr size_t smem_bytes() {
  return (size_t)STAGES * (A_BYTES * (DUAL ? 2 : 1) + NT * 128) + 1024;
}

template <int NT, bool DUAL, int STAGES>
cudaError_t launch_one(int* status, const TcGemm& g, cudaStream_t st) {
  dim3 grid(g.N / 128, (g.M + NT - 1) / NT, g.splits > 0 ? g.splits : 1);
  k_gemm_tc<NT, DUAL, STAGES><<<grid, 288, smem_bytes<NT, DUAL, STAGES>(), st>>>(status, g);
  return cudaGetLastError();
}

template <int NT, bool DUAL, int STAGES>
cudaError_t setup_one() {
  return cudaFuncSetAttribute(k_gemm_tc<NT, DUAL, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)smem_bytes<NT, DUAL, STAGES>());
}

}  // namespace

cudaError_t tc_gemm_setup() {
  cudaError_t e;
  if ((e = setup_one<64, false, 6>()) != cudaSuccess) return e;
  if ((e = setup_one<64, true, 4>()) != cudaSuccess) return e;
  if ((e = setup_one<128, false, 5>()) != cudaSuccess) return e;
  if ((e = setup_one<128, true, 4>()) != cudaSuccess) return e;
  if ((e = setup_one<256, false, 4>()) != cudaSuccess) return e;
  if ((e = setup_one<256, true, 3>()) != cudaSuccess) return e;
  return cudaSuccess;
}

cudaError_t launch_tc_gemm(int* status, const TcGemm& g, int nt, cudaStream_t st) {
  const bool dual = g.epi == TC_GEGLU;
  if (nt == 64) return dual ? launch_one<64, true, 4>(status, g, st) : launch_one<64, false, 6>(status, g, st);
  if (nt == 128) return dual ? launch_one<128, true, 4>(status, g, st) : launch_one<128, false, 5>(status, g, st);
  return dual ? launch_one<256, true, 3>(status, g, st) : launch_one<256, false, 4>(status, g, st);
}

}  // namespace phyai
