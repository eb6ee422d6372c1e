// Large-batch bf16 GEMM on CTA pairs: tcgen05.mma.cta_group::2, persistent, epilogue overlapped with
// the next tile's main loop.
//
// Orientation ("tokens on the M axis"): a pair of CTAs (a cluster of two, one per SM of a TPC) computes
// a 256-token x 256-channel tile.  Each CTA stages its own 128 token rows (A operand) and one 128-channel
// weight block (its half of the B operand); the leader CTA issues one M = 256, N = 256 MMA per K = 16
// that reads both CTAs' shared memory and writes each CTA's 128 x 256 accumulator in that CTA's tensor
// memory.  Per 64-wide k-chunk a CTA therefore fetches 32 KB for 512 tensor clocks -- the 64 bytes per
// clock one SM's L2 port delivers -- and the accumulator takes 256 of the 512 TMEM columns, so two
// accumulator stages fit and the epilogue of tile i runs under the main loop of tile i + 1.
//
// Both operands are K-major with the 128-byte swizzle and come in 128-row blocks of 16 KB: the packed
// weight blocks and the tiled bf16 activations of the other GEMM kernel are used unchanged, and every
// load is a 1-D bulk copy.
//
// An epilogue thread owns one token row (TMEM lane) and walks channel columns, so per-token work needs no
// cross-thread exchange: GeGLU reads gate and up of a channel from two columns of its own lane (the pair's
// first CTA stages the gate block, the second the up block).  Results are transposed per warp through a
// small shared-memory block so that global accesses cover whole 128-byte lines.
//
// Warps (576 threads): 0-3 and 4-7 epilogue (TMEM lane quarter = warp % 4, column half = warp / 4),
// 8 TMEM owner + MMA issuer (leader CTA only issues), 9 relay (second CTA: forwards "stage landed" to the
// leader), 10-17 bulk-copy producers.  Synchronisation between the two CTAs uses cluster-scope mbarrier
// arrives and tcgen05.commit multicast; every wait is bounded, and on expiry the CTA raises the status
// word, stops issuing and drains to the common exit (cluster barrier, then TMEM release).
#include "kernels.h"
#include "ptx.cuh"
#include "tc.cuh"

namespace phyai {
namespace {

constexpr int BLK = 128 * 128;       // one operand block: 128 rows x 64 k (bf16)
constexpr int STAGE2 = 2 * BLK;      // per CTA and stage: its token rows + its weight block
constexpr int NSTAGE = 5;
constexpr int STG_ROW = 144;         // staging row pitch in bytes (128 + 16: conflict-free 16-byte accesses)
constexpr int STG_BYTES = 32 * STG_ROW;   // per epilogue warp: 32 rows
constexpr int NPROD2 = 8;
constexpr int THREADS2 = 576;
constexpr int ACC_COLS = 256;
// A producer warp issues every (NPROD2 / 2)-th k-chunk.  Its "stage is free" wait is a parity wait, which is
// only meaningful while the warp is less than one full ring ahead of the barrier's phase: the step between
// a warp's consecutive k-chunks must not exceed the ring depth.
static_assert(NPROD2 / 2 <= NSTAGE, "producer stride exceeds the stage ring");

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on the barrier at the same shared-memory offset in CTA `cta` of the cluster.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar, uint32_t cta) {
  asm volatile(
      "{\n.reg .b32 ra;\n"
      "mapa.shared::cluster.u32 ra, %0, %1;\n"
      "mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra];\n}" ::"r"(bar),
      "r"(cta)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D (both CTAs' TMEM, 128 rows each) (+)= A (both CTAs' rows) * B (both CTAs' column halves)^T
__device__ __forceinline__ void umma2_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on `bar` in both CTAs of the pair once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"(mask)
               : "memory");
}
template <int BAR>
__device__ __forceinline__ void half_sync() { asm volatile("bar.sync %0, 128;" ::"n"(BAR) : "memory"); }

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS2, 1) k_gemm_pair(int* status, const TcGemm g) {
  constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((256u >> 4) << 24);

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[NSTAGE], bar_empty[NSTAGE], bar_peer_full[NSTAGE];
  __shared__ __align__(8) uint64_t bar_acc_full[2], bar_acc_empty[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag, skip_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();          // 0 = leader of the pair
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const bool geglu = g.epi == TC_GEGLU;
  const int KC = g.K >> 6;
  const int m_tiles = (g.M + 255) >> 8;
  const int n_tiles = geglu ? g.N >> 7 : g.N >> 8;

  if (threadIdx.x == 0) {
    skip_flag = status_set(status) ? 1 : 0;
    abort_flag = 0;
    for (int s = 0; s < NSTAGE; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 2);
      mbar_init(smem_u32(&bar_empty[s]), 1);
      mbar_init(smem_u32(&bar_peer_full[s]), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&bar_acc_full[s]), 1);
      mbar_init(smem_u32(&bar_acc_empty[s]), 4);   // two column halves in each of the two CTAs
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    tmem_alloc2(smem_u32(&tmem_slot), 512);
    tc_fence_before();
  }
  __syncthreads();
  cluster_sync_all();                            // the peer's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  const WaitCtx wc{status, &abort_flag, g.wait_limit};
  const int total = skip_flag ? 0 : m_tiles * n_tiles;
  const int my_tiles = pair < total ? (total - pair + n_pairs - 1) / n_pairs : 0;
  const int n_it = my_tiles * KC;                // k-chunks this pair walks
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;

  if (warp >= 10) {
    // ---------------- producers: copy id = 2 * it + {0: token rows, 1: weight block}, dealt to 8 warps ----
    if (lane == 0) {
      const uint8_t* X = reinterpret_cast<const uint8_t*>(g.X);
      const uint8_t* W = reinterpret_cast<const uint8_t*>((geglu && rank == 1) ? g.W2 : g.W);
      for (int id = warp - 10; id < 2 * n_it; id += NPROD2) {
        const int it = id >> 1, c = id & 1;
        const int tl = it / KC, kc = it - tl * KC;
        const int tile = pair + tl * n_pairs;
        const int mt = tile % m_tiles, nt = tile / m_tiles;
        const int s = it % NSTAGE;
        const uint32_t ph = (uint32_t)(it / NSTAGE) & 1u;
        if (!mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc)) break;   // stop issuing copies once aborted
        const uint32_t full = smem_u32(&bar_full[s]);
        const uint32_t dst = tiles + (uint32_t)s * STAGE2 + (uint32_t)c * BLK;
        const uint8_t* src;
        if (c == 0) {
          src = X + ((size_t)kc * g.rows_pad + (size_t)mt * 256 + rank * 128) * 128;
        } else {
          const int wt = geglu ? nt : nt * 2 + (int)rank;
          src = W + ((size_t)wt * KC + kc) * BLK;
        }
        mbar_expect_tx(full, BLK);
        bulk_g2s(dst, src, BLK, full);
      }
    }
  } else if (warp == 9) {
    // ---------------- relay (second CTA): tell the leader that this CTA's stage has landed ----------------
    if (rank == 1 && lane == 0) {
      for (int it = 0; it < n_it; ++it) {
        const int s = it % NSTAGE;
        if (!mbar_wait(smem_u32(&bar_full[s]), (uint32_t)(it / NSTAGE) & 1u, wc)) break;
        mbar_arrive_remote(smem_u32(&bar_peer_full[s]), 0);
      }
    }
  } else if (warp == 8) {
    // ---------------- MMA issuer (leader CTA; whole warp in the loop, one elected lane issues) -----------
    if (rank == 0) {
      int it = 0;
      for (int tl = 0; tl < my_tiles; ++tl) {
        const int as = tl & 1;
        // the epilogues of both CTAs have drained this accumulator stage (first use passes at once)
        bool ok = mbar_wait(smem_u32(&bar_acc_empty[as]), ((uint32_t)(tl >> 1) & 1u) ^ 1u, wc);
        tc_fence_after();
        const uint32_t d = tmem_base + (uint32_t)as * ACC_COLS;
        for (int kc = 0; kc < KC; ++kc, ++it) {
          const int s = it % NSTAGE;
          const uint32_t ph = (uint32_t)(it / NSTAGE) & 1u;
          ok = mbar_wait(smem_u32(&bar_full[s]), ph, wc) && ok;
          ok = mbar_wait(smem_u32(&bar_peer_full[s]), ph, wc) && ok;
          tc_fence_after();
          const uint32_t a0 = tiles + (uint32_t)s * STAGE2;
          const uint64_t da = make_desc(a0), db = make_desc(a0 + BLK);
          if (__all_sync(0xffffffffu, ok)) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
              if (elect_one()) umma2_bf16(d, da + 2 * k, db + 2 * k, IDESC, (kc > 0 || k > 0) ? 1u : 0u);
          }
          if (elect_one()) umma2_commit_both(smem_u32(&bar_empty[s]));   // frees the stage in both CTAs
          __syncwarp();
        }
        if (elect_one()) umma2_commit_both(smem_u32(&bar_acc_full[as]));
        __syncwarp();
      }
    }
  } else {
    // ---------------- epilogue (warps 0-7): TMEM -> registers -> shared staging -> global ------------------
    // A thread reads its token row from TMEM; the warp then transposes each 32-row block through a padded
    // shared-memory buffer so that every global access covers whole 128-byte lines (4 rows x 128 bytes per
    // instruction) instead of 16 bytes in each of 32 rows.
    const int q = warp & 3, ch = warp >> 2;       // TMEM lane quarter, column half
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    const uint32_t stg = tiles + (uint32_t)NSTAGE * STAGE2 + (uint32_t)warp * STG_BYTES;   // this warp's staging block
    const int sr = lane >> 3, sc = lane & 7;      // staging read: rows sr, sr + 4, ...; 16-byte column sc
    for (int tl = 0; tl < my_tiles; ++tl) {
      const int tile = pair + tl * n_pairs;
      const int mt = tile % m_tiles, nt = tile / m_tiles;
      const int as = tl & 1;
      const bool ok = mbar_wait(smem_u32(&bar_acc_full[as]), (uint32_t)(tl >> 1) & 1u, wc);
      tc_fence_after();
      const int tok0 = mt * 256 + (int)rank * 128 + q * 32;   // first token row of this warp
      const int tok = tok0 + lane;
      const uint32_t acc = tmem_base + (uint32_t)as * ACC_COLS + lane_addr;
      if (geglu) {
        // columns [0, 128) = gate, [128, 256) = up of channels nt * 128 ..; this half takes 64 of them, which
        // are one 128-byte row of the down projection's tiled input (16-byte chunks XOR-swizzled by the row)
        const int cb = ch * 64;
#pragma unroll 1
        for (int c0 = 0; c0 < 64; c0 += 16) {
          float vg[16], vu[16];
          tmem_ld16(acc + (uint32_t)(cb + c0), vg);
          tmem_ld16(acc + (uint32_t)(128 + cb + c0), vu);
          const int n = nt * 128 + cb + c0;
          uint32_t w[8];
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            const float g0 = g.scale ? vg[j] * __ldg(g.scale + n + j) : vg[j];
            const float g1 = g.scale ? vg[j + 1] * __ldg(g.scale + n + j + 1) : vg[j + 1];
            const float u0 = g.scale2 ? vu[j] * __ldg(g.scale2 + n + j) : vu[j];
            const float u1 = g.scale2 ? vu[j + 1] * __ldg(g.scale2 + n + j + 1) : vu[j + 1];
            w[j >> 1] = pack2(gelu_fast(g0, g.gelu_exact) * u0, gelu_fast(g1, g.gelu_exact) * u1);
          }
          const int c8 = c0 >> 3;
          st_shared_v4(stg + (uint32_t)lane * STG_ROW + (uint32_t)(((c8) ^ (tok & 7)) << 4), w[0], w[1], w[2], w[3]);
          st_shared_v4(stg + (uint32_t)lane * STG_ROW + (uint32_t)(((c8 + 1) ^ (tok & 7)) << 4), w[4], w[5], w[6], w[7]);
        }
        __syncwarp();
        __nv_bfloat16* dst = g.out_tiled + ((size_t)(nt * 2 + ch) * g.rows_pad + tok0) * 64 + sc * 8;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int r = k * 4 + sr;
          const uint4 val = ld_shared_v4(stg + (uint32_t)r * STG_ROW + (uint32_t)sc * 16);
          if (ok && tok0 + r < g.M) *reinterpret_cast<uint4*>(dst + (size_t)r * 64) = val;
        }
        __syncwarp();
      } else {
        const int cb = ch * 128;
#pragma unroll 1
        for (int c0 = 0; c0 < 128; c0 += 32) {
          float v[32];
          tmem_ld16(acc + (uint32_t)(cb + c0), v);
          tmem_ld16(acc + (uint32_t)(cb + c0 + 16), v + 16);
          const int n = nt * 256 + cb + c0;          // packed output channel of v[0]
          if (g.scale) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] *= __ldg(g.scale + n + j);
          }
#pragma unroll
          for (int j = 0; j < 8; ++j)
            st_shared_v4(stg + (uint32_t)lane * STG_ROW + (uint32_t)j * 16, __float_as_uint(v[4 * j]), __float_as_uint(v[4 * j + 1]),
                         __float_as_uint(v[4 * j + 2]), __float_as_uint(v[4 * j + 3]));
          __syncwarp();
          // this lane now handles columns n + 4 * sc .. + 3 of rows sr, sr + 4, ...
          const int np = n + 4 * sc;
          const int no = (g.epi == TC_STORE && g.perm_dh && np < g.perm_end) ? qkv_packed_to_channel(np, g.perm_dh) : np;
          float* optr = g.out_f32 + (size_t)tok0 * g.ldo + no;
          if (g.epi == TC_RESID) {
            float4 gt = make_float4(1.f, 1.f, 1.f, 1.f);
            if (g.gate) gt = __ldg(reinterpret_cast<const float4*>(g.gate + np));
            float4 old[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const int r = k * 4 + sr;
              old[k] = (ok && tok0 + r < g.M) ? *reinterpret_cast<const float4*>(optr + (size_t)r * g.ldo)
                                             : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const int r = k * 4 + sr;
              const uint4 u = ld_shared_v4(stg + (uint32_t)r * STG_ROW + (uint32_t)sc * 16);
              old[k].x += gt.x * __uint_as_float(u.x), old[k].y += gt.y * __uint_as_float(u.y);
              old[k].z += gt.z * __uint_as_float(u.z), old[k].w += gt.w * __uint_as_float(u.w);
              if (ok && tok0 + r < g.M) *reinterpret_cast<float4*>(optr + (size_t)r * g.ldo) = old[k];
            }
          } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const int r = k * 4 + sr;
              const uint4 u = ld_shared_v4(stg + (uint32_t)r * STG_ROW + (uint32_t)sc * 16);
              if (ok && tok0 + r < g.M) *reinterpret_cast<uint4*>(optr + (size_t)r * g.ldo) = u;
            }
          }
          __syncwarp();
        }
      }
      tc_fence_before();
      if (ch == 0) half_sync<1>(); else half_sync<2>();
      if ((threadIdx.x & 127) == 0) mbar_arrive_remote(smem_u32(&bar_acc_empty[as]), 0);   // to the leader
    }
  }

  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    // give any bulk copy still in flight time to land before shared memory is released
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  cluster_sync_all();                            // neither CTA leaves (or frees TMEM) while the other may still signal it
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc2(tmem_base, 512);
  }
}

constexpr size_t PAIR_SMEM = (size_t)NSTAGE * STAGE2 + 8 * STG_BYTES + 1024;

}  // namespace

cudaError_t tc_gemm_pair_setup() {
  return cudaFuncSetAttribute(k_gemm_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PAIR_SMEM);
}

bool tc_gemm_pair_supported(const TcGemm& g) {
  if (g.epi != TC_STORE && g.epi != TC_RESID && g.epi != TC_GEGLU) return false;
  if (g.splits > 1 || g.K % 64 || g.rows_pad % 256) return false;
  return g.epi == TC_GEGLU ? g.N % 128 == 0 : g.N % 256 == 0;
}

cudaError_t launch_tc_gemm_pair(int* status, const TcGemm& g, int n_sm, cudaStream_t st) {
  const int tiles = ((g.M + 255) / 256) * (g.epi == TC_GEGLU ? g.N / 128 : g.N / 256);
  int pairs = n_sm / 2;
  if (pairs > tiles) pairs = tiles;
  if (pairs < 1) pairs = 1;
  k_gemm_pair<<<2 * pairs, THREADS2, PAIR_SMEM, st>>>(status, g);
  return cudaGetLastError();
}

}  // namespace phyai
