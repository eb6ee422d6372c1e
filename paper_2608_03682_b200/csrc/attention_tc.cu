// Suffix -> (prefix U suffix) attention on the tcgen05 tensor cores, for large batches.
//
// One CTA takes the suffix rows of two query heads that share a kv head (2 x 64 padded rows = the 128
// rows of one MMA) and walks all key tiles of its request:
//   S = Q K^T      tcgen05.mma, M = 128, N = 64 keys, K = head_dim, fp32 accumulator in TMEM
//   softmax        one thread per row reads its S row from TMEM (no shuffles), online max / sum in the
//                  log2 domain, writes P (bf16) to shared memory as the next MMA's A operand
//   O += P V       tcgen05.mma, M = 128, N = head_dim, K = 64 keys, accumulator stays in TMEM; V is used
//                  as an MN-major B operand, so K and V tiles share one shared-memory layout and loader
// K/V tiles (64 keys) are double buffered and staged with 16-byte cp.async into the 128-byte-swizzled
// block layout the MMA descriptors expect.  The O accumulator is rescaled only when a row's running
// maximum grows by more than 2^8 (otherwise the old maximum is kept, which is exact algebra and costs
// nothing), so the TMEM round trip of the correction is rare.
//
// Warps: 0-3 load K/V (and build Q and the suffix tile), 4 issues the MMAs (whole warp in the loop, one
// elected lane issues), 5-8 softmax / correction / output (TMEM lane quarter = warp % 4).
// All waits are bounded; on expiry the CTA raises the status word and drains.
#include "attention.cuh"
#include "tc.cuh"

namespace phyai {
namespace {

constexpr int KTC = 64;          // keys per tile
constexpr int BAR_LOAD = 1;      // named barrier of the 4 loader warps
constexpr int BAR_SOFT = 2;      // named barrier of the 4 softmax warps
constexpr float RESCALE_THRESHOLD = 8.0f;   // log2 units

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
      "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
      "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
      "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_local(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// MN-major operand, 128-byte swizzle: 64 contiguous elements (128 bytes) along N per row, 8-row groups
// along K `sbo` bytes apart, 64-element groups along N `lbo` bytes apart.
__device__ __forceinline__ uint64_t make_desc_mn(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

template <int DH>
__global__ void __launch_bounds__(288, 1) k_attn_tc(const AttnArgs a) {
  constexpr int NB = DH / 64;                 // 64-element blocks along head_dim
  constexpr int Q_BYTES = 128 * DH * 2;       // NB blocks of [128 rows x 128 B]
  constexpr int KV_BYTES = KTC * DH * 2;      // NB blocks of [64 keys x 128 B]
  constexpr int KV_BLOCK = KTC * 128;
  constexpr int P_BYTES = 128 * KTC * 2;      // one block [128 rows x 64 keys]
  constexpr int COLS = 512;                   // S at columns [0, 64), O at [64, 64 + DH)
  constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(KTC >> 3) << 17) | ((128u >> 4) << 24);
  constexpr uint32_t IDESC_PV =
      (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((128u >> 4) << 24);

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t kv_full[2], kv_free[2], s_full, s_free, p_full, pv_done;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag, skip_flag;

  const Dims& d = a.d;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int hp = blockIdx.x, b = blockIdx.y;
  const int head0 = hp * 2;
  const int hk = head0 / (d.Hq / d.Hkv);
  const int S = d.S;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t Qs = base, Ks = Qs + Q_BYTES, Vs = Ks + 2 * KV_BYTES, Ps = Vs + 2 * KV_BYTES;
  uint8_t* Ps_ptr = smem_raw + (Ps - smem_u32(smem_raw));

  if (tid == 0) {
    skip_flag = status_set(a.status) ? 1 : 0;
    abort_flag = 0;
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&kv_full[i]), 1);
      mbar_init(smem_u32(&kv_free[i]), 1);
    }
    mbar_init(smem_u32(&s_full), 1);
    mbar_init(smem_u32(&s_free), 1);
    mbar_init(smem_u32(&p_full), 1);
    mbar_init(smem_u32(&pv_done), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (skip_flag) return;
  if (warp == 4) {
    tmem_alloc(smem_u32(&tmem_slot), COLS);
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + KTC;
  const WaitCtx wc{a.status, &abort_flag, a.wait_limit};

  const Request r = *a.rq;
  const int p0 = r.cu_lens[b], P = r.cu_lens[b + 1] - p0;
  const int Tp = (P + KTC - 1) / KTC;
  const int T = Tp + 1;                       // the suffix (<= 64 keys) is the last tile
  constexpr int half = DH / 2;

  if (warp < 4) {
    // =========================== loaders ==========================================================
    const int lt = tid;   // 0..127
    const uint8_t* Kg = reinterpret_cast<const uint8_t*>(r.prefix_kv) +
                        (((size_t)(a.layer * 2 + 0) * r.kv_tokens + p0) * d.Hkv + hk) * (DH * 2);
    const uint8_t* Vg = reinterpret_cast<const uint8_t*>(r.prefix_kv) +
                        (((size_t)(a.layer * 2 + 1) * r.kv_tokens + p0) * d.Hkv + hk) * (DH * 2);
    const size_t kv_stride = (size_t)d.Hkv * DH * 2;
    // ---- Q: rotate, scale, round to bf16 into the [block][row][128 B] swizzled image ----
    const float qscale = rsqrtf((float)DH);
    for (int idx = lt; idx < 128 * (half / 4); idx += 128) {
      const int row = idx / (half / 4), j = (idx % (half / 4)) * 4;   // row = head_local * 64 + i
      const int hl = row >> 6, i = row & 63;
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
      auto put = [&](int col, float4 v) {   // 4 consecutive columns of `row`
        const int blk = col >> 6, c = (col & 63) >> 3;
        const uint32_t addr = Qs + (uint32_t)blk * (128 * 128) + (uint32_t)row * 128 + (uint32_t)((c ^ (row & 7)) << 4) +
                              (uint32_t)(col & 7) * 2;
        asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(addr), "r"(pack_bf16(v.x * qscale, v.y * qscale)),
                     "r"(pack_bf16(v.z * qscale, v.w * qscale))
                     : "memory");
      };
      put(j, lo);
      put(j + half, hi);
    }
    for (int t = 0; t < T; ++t) {
      const int buf = t & 1;
      const uint32_t ph = (uint32_t)(t >> 1) & 1u;
      if (t >= 2) mbar_wait(smem_u32(&kv_free[buf]), ph ^ 1u, wc);   // PV of tile t-2 has read this buffer
      const uint32_t kb = Ks + (uint32_t)buf * KV_BYTES, vb = Vs + (uint32_t)buf * KV_BYTES;
      if (t < Tp) {
        const int rows = min(KTC, P - t * KTC);
        for (int idx = lt; idx < KTC * (DH / 8); idx += 128) {
          const int row = idx / (DH / 8), c = idx % (DH / 8);
          const bool ok = row < rows;
          const size_t g = (size_t)(t * KTC + (ok ? row : 0)) * kv_stride + (size_t)c * 16;
          const uint32_t o = (uint32_t)(c >> 3) * KV_BLOCK + (uint32_t)row * 128 + (uint32_t)(((c & 7) ^ (row & 7)) << 4);
          cp_async16(kb + o, Kg + g, ok ? 16u : 0u);
          cp_async16(vb + o, Vg + g, ok ? 16u : 0u);
        }
        cp_async_commit();
        cp_async_wait<0>();
      } else {
        // suffix tile: rotate this request's own keys, round K and V to bf16
        for (int idx = lt; idx < KTC * (half / 4); idx += 128) {
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
          auto put = [&](uint32_t tb, int col, float4 v) {
            const uint32_t addr = tb + (uint32_t)(col >> 6) * KV_BLOCK + (uint32_t)js * 128 +
                                  (uint32_t)((((col & 63) >> 3) ^ (js & 7)) << 4) + (uint32_t)(col & 7) * 2;
            asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(addr), "r"(pack_bf16(v.x, v.y)), "r"(pack_bf16(v.z, v.w))
                         : "memory");
          };
          put(kb, j, klo), put(kb, j + half, khi), put(vb, j, vlo), put(vb, j + half, vhi);
        }
      }
      fence_async_smem();                  // these generic-proxy writes are read by the tensor core
      group_sync<BAR_LOAD, 128>();
      if (lt == 0) mbar_arrive_local(smem_u32(&kv_full[buf]));
    }
  } else if (warp == 4) {
    // =========================== MMA issuer ========================================================
    for (int t = 0; t < T; ++t) {
      const int buf = t & 1;
      const uint32_t ph = (uint32_t)(t >> 1) & 1u;
      bool ok = mbar_wait(smem_u32(&kv_full[buf]), ph, wc);
      if (t > 0) ok = mbar_wait(smem_u32(&s_free), (uint32_t)(t - 1) & 1u, wc) && ok;   // softmax has read S of t-1
      tc_fence_after();
      const uint32_t kb = Ks + (uint32_t)buf * KV_BYTES, vb = Vs + (uint32_t)buf * KV_BYTES;
      const bool go = __all_sync(0xffffffffu, ok);
      // ---- S = Q K^T ----
      if (go) {
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {
          const uint64_t da = make_desc(Qs + (uint32_t)(kk >> 2) * (128 * 128) + (uint32_t)(kk & 3) * 32);
          const uint64_t db = make_desc(kb + (uint32_t)(kk >> 2) * KV_BLOCK + (uint32_t)(kk & 3) * 32);
          if (elect_one()) umma_bf16(tmem_s, da, db, IDESC_S, kk > 0 ? 1u : 0u);
        }
      }
      if (elect_one()) umma_commit(smem_u32(&s_full));
      __syncwarp();
      // ---- O += P V ----
      ok = mbar_wait(smem_u32(&p_full), (uint32_t)t & 1u, wc);
      tc_fence_after();
      if (__all_sync(0xffffffffu, ok) && go) {
#pragma unroll
        for (int kj = 0; kj < KTC / 16; ++kj) {
          const uint64_t da = make_desc(Ps + (uint32_t)kj * 32);
          const uint64_t db = make_desc_mn(vb + (uint32_t)kj * (16 * 128), KV_BLOCK, 1024);
          if (elect_one()) umma_bf16(tmem_o, da, db, IDESC_PV, (t > 0 || kj > 0) ? 1u : 0u);
        }
      }
      if (elect_one()) {
        umma_commit(smem_u32(&kv_free[buf]));
        umma_commit(smem_u32(&pv_done));
      }
      __syncwarp();
    }
  } else {
    // =========================== softmax / correction / output =====================================
    const int st = tid - 160;                 // 0..127
    const int q = warp & 3;
    const int row = q * 32 + lane;            // accumulator row = TMEM lane
    const int hl = row >> 6, i = row & 63;
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    float m = -INFINITY, l = 0.f;
    const bool causal_row = d.block_causal && d.ns && i == 0;
    for (int t = 0; t < T; ++t) {
      const bool ok = mbar_wait(smem_u32(&s_full), (uint32_t)t & 1u, wc);
      tc_fence_after();
      const int valid = t < Tp ? min(KTC, P - t * KTC) : S;
      float s[KTC];
#pragma unroll
      for (int c = 0; c < KTC; c += 16) tmem_ld16(tmem_s + lane_addr + (uint32_t)c, s + c);
      tc_fence_before();
      group_sync<BAR_SOFT, 128>();
      if (st == 0) mbar_arrive_local(smem_u32(&s_free));     // S may be overwritten by the next tile
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < KTC; ++c) {
        bool vis = c < valid;
        if (causal_row && t >= Tp && c != 0) vis = false;   // state token sees, of the suffix, only itself
        s[c] = vis ? s[c] * LOG2E : -INFINITY;
        mx = fmaxf(mx, s[c]);
      }
      // running maximum: keep the old one unless the new exceeds it by more than the threshold
      float m_new = m;
      if (mx > m + RESCALE_THRESHOLD || m == -INFINITY) m_new = fmaxf(m, mx);
      const bool rescale = m_new != m && m != -INFINITY;
      const float corr = rescale ? exp2f(m - m_new) : 1.0f;
      const float sub = m_new == -INFINITY ? 0.f : m_new;
      float rs = 0.f;
      // the previous tile's P V must have finished before P is overwritten (and before O is touched)
      bool okp = true;
      if (t > 0) okp = mbar_wait(smem_u32(&pv_done), (uint32_t)(t - 1) & 1u, wc);
      tc_fence_after();
#pragma unroll
      for (int c8 = 0; c8 < KTC / 8; ++c8) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float p0 = exp2f(s[c8 * 8 + 2 * e] - sub), p1 = exp2f(s[c8 * 8 + 2 * e + 1] - sub);
          rs += p0 + p1;
          w[e] = pack_bf16(p0, p1);
        }
        *reinterpret_cast<uint4*>(Ps_ptr + (size_t)row * 128 + (size_t)((c8 ^ (row & 7)) << 4)) =
            make_uint4(w[0], w[1], w[2], w[3]);
      }
      l = l * corr + rs;
      m = m_new;
      if (__any_sync(0xffffffffu, rescale)) {     // rare: rescale this warp's 32 accumulator rows
#pragma unroll 1
        for (int c = 0; c < DH; c += 16) {
          float o[16];
          tmem_ld16(tmem_o + lane_addr + (uint32_t)c, o);
#pragma unroll
          for (int e = 0; e < 16; ++e) o[e] *= corr;
          tmem_st16(tmem_o + lane_addr + (uint32_t)c, o);
        }
        tmem_st_wait();
      }
      tc_fence_before();
      fence_async_smem();
      group_sync<BAR_SOFT, 128>();
      if (st == 0) mbar_arrive_local(smem_u32(&p_full));
      (void)ok;
      (void)okp;
    }
    // ---- output: O / l -> bf16 ----
    const bool okf = __all_sync(0xffffffffu, mbar_wait(smem_u32(&pv_done), (uint32_t)(T - 1) & 1u, wc));
    tc_fence_after();
    {
      const bool wr = okf && i < S;             // the TMEM loads stay warp-uniform; only the stores are predicated
      const float inv = 1.0f / l;
      const int orow = b * S + (i < S ? i : 0), head = head0 + hl;
#pragma unroll 1
      for (int c = 0; c < DH; c += 16) {
        float o[16];
        tmem_ld16(tmem_o + lane_addr + (uint32_t)c, o);
        const uint4 lo = make_uint4(pack_bf16(o[0] * inv, o[1] * inv), pack_bf16(o[2] * inv, o[3] * inv),
                                    pack_bf16(o[4] * inv, o[5] * inv), pack_bf16(o[6] * inv, o[7] * inv));
        const uint4 hi = make_uint4(pack_bf16(o[8] * inv, o[9] * inv), pack_bf16(o[10] * inv, o[11] * inv),
                                    pack_bf16(o[12] * inv, o[13] * inv), pack_bf16(o[14] * inv, o[15] * inv));
        if (wr) {
          *reinterpret_cast<uint4*>(a.out + out_index(orow, head * DH + c, a.rows_pad, d.Nq)) = lo;
          *reinterpret_cast<uint4*>(a.out + out_index(orow, head * DH + c + 8, a.rows_pad, d.Nq)) = hi;
        }
      }
    }
    tc_fence_before();
  }

  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem_base, COLS);
  }
}

template <int DH>
constexpr size_t attn_tc_smem() {
  return 1024 + (size_t)128 * DH * 2 + 4 * (size_t)KTC * DH * 2 + (size_t)128 * KTC * 2;
}

}  // namespace

bool attention_tc_supported(const Dims& d) {
  return d.dh == 256 && d.S <= 64 && d.Hq % 2 == 0 && (d.Hq / d.Hkv) % 2 == 0;
}

cudaError_t launch_attention_tc(const Request* rq, int* status, const float* qkv, const float2* rope, int layer,
                                __nv_bfloat16* out_tiled, int rows_pad, const Dims& d, int batch, unsigned wait_limit,
                                cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(k_attn_tc<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)attn_tc_smem<256>());
    if (e != cudaSuccess) return e;
    configured = true;
  }
  AttnArgs a{};
  a.rq = rq, a.status = status, a.qkv = qkv, a.rope = rope, a.layer = layer, a.out = out_tiled, a.rows_pad = rows_pad;
  a.num_splits = 1, a.d = d, a.wait_limit = wait_limit;
  dim3 grid(d.Hq / 2, batch);
  k_attn_tc<256><<<grid, 288, attn_tc_smem<256>(), st>>>(a);
  return cudaGetLastError();
}

}  // namespace phyai
