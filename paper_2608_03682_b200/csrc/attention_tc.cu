// Suffix -> (prefix U suffix) attention on the tcgen05 tensor cores, for calls with two or more requests.
//
// One CTA takes the suffix rows of two query heads that share a kv head (2 x 64 padded rows = the 128
// rows of one MMA) and walks all key tiles of its request:
//   S = Q K^T      tcgen05.mma, M = 128, N = 64 keys, K = head_dim; Q sits in tensor memory (A operand), K in
//                  shared memory; fp32 accumulator in TMEM, two buffers
//   softmax        one thread per row reads its S row from TMEM (no shuffles), online max / sum in the log2
//                  domain, writes P (bf16 pairs) over the first half of the S buffer it has just read
//   O += P V       tcgen05.mma, M = 128, N = head_dim, K = 64 keys; P is the tensor-memory A operand, V an
//                  MN-major B operand in shared memory (K and V tiles share one layout and loader code);
//                  the accumulator stays in TMEM
// TMEM columns: S / P buffers [0, 128), O [128, 384), Q [384, 512).  The tensor pipe executes one thread's MMAs
// in issue order, which is what lets P alias S: S(t + 2) is issued after P(t) V(t).
// K and V tiles (64 keys) stream through two three-deep rings, each filled by its own pair of warps with 16-byte
// cp.async into the 128-byte-swizzled block layout the MMA descriptors expect.  The suffix keys are tile 0; the
// prefix tiles follow.  Q and the suffix K / V arrive as bf16, already rotated (q also scaled), from the QKV
// projection's epilogue.  The O accumulator is rescaled only when a row's running maximum grows by more than 2^8
// (otherwise the old maximum is kept, which is exact algebra and costs nothing), so the TMEM round trip of the
// correction is rare.
//
// Warps: 0-1 load K, 2-3 load V, 4 issues the MMAs (whole warp in the loop, one elected lane issues), 5-8 Q into
// TMEM, softmax / correction / output (TMEM lane quarter = warp % 4).
// All waits are bounded; on expiry the CTA raises the status word and drains.
#include "attention.cuh"
#include "tc.cuh"

namespace phyai {
namespace {

constexpr int KTC = 64;          // keys per tile
constexpr int NKV = 3;           // K and V tile buffers each
constexpr int BAR_LOAD = 1;      // named barrier of the 2 K loader warps
constexpr int BAR_SOFT = 2;      // named barrier of the 4 softmax warps (3 = the V loader warps)
constexpr int BAR_QSTAGE = 4;    // softmax warps (arrive) -> V loader warps (sync): the Q staging area is free
constexpr float RESCALE_THRESHOLD = 8.0f;   // log2 units

template <int DH>
__global__ void __launch_bounds__(288, 1) k_attn_tc(const AttnArgs a) {
  constexpr int KV_BYTES = KTC * DH * 2;      // DH/64 blocks of [64 keys x 128 B]
  constexpr int KV_BLOCK = KTC * 128;
  constexpr int COLS = 512;                   // S / P (two buffers) at columns [0, 128), O at [128, 384), Q at [384, 512)
  constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(KTC >> 3) << 17) | ((128u >> 4) << 24);
  constexpr uint32_t IDESC_PV =
      (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((128u >> 4) << 24);

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t k_full[NKV], v_full[NKV], p_full[2], pv_done[2], s_full[2], q_full, fin_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag, skip_flag;

  const Dims& d = a.d;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int hp = blockIdx.x;
  const int b = a.order ? a.order[blockIdx.y] : (int)blockIdx.y;   // longest requests first
  const int head0 = hp * 2;
  const int hk = head0 / (d.Hq / d.Hkv);
  const int S = d.S;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t Ks = base, Vs = Ks + NKV * KV_BYTES;

  unsigned long long* const trc = a.trace ? a.trace + (size_t)((blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) * 16 : nullptr;
  if (tid == 0) trace_stamp(trc, 0);
  // Programmatic dependent launch: barriers and tensor memory are set up while the kernel before this one (the q|k|v
  // projection) still runs; the first access to anything it wrote comes after pdl_wait().
  pdl_launch_dependents();
  if (tid == 0) {
    abort_flag = 0;
    for (int i = 0; i < NKV; ++i) {
      mbar_init(smem_u32(&k_full[i]), 1);
      mbar_init(smem_u32(&v_full[i]), 1);
    }
    mbar_init(smem_u32(&q_full), 1);
    mbar_init(smem_u32(&fin_bar), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&p_full[i]), 1);
      mbar_init(smem_u32(&pv_done[i]), 1);
      mbar_init(smem_u32(&s_full[i]), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    tmem_alloc(smem_u32(&tmem_slot), COLS);
    tc_fence_before();
  }
  const WaitCtx wc{a.status, &abort_flag, a.wait_limit};
  __syncthreads();                             // barriers initialised, the TMEM base address published
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  pdl_wait();
  if (tid == 0) {
    trace_stamp(trc, 1);
    skip_flag = status_set(a.status) ? 1 : 0;
  }
  __syncthreads();
  if (skip_flag) {
    if (warp == 4) tmem_dealloc(tmem_base, COLS);
    return;
  }
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + 2 * KTC, tmem_q = tmem_base + 2 * KTC + DH;

  const Request r = *a.rq;
  const int p0 = r.cu_lens[b], P = r.cu_lens[b + 1] - p0;
  const int Tp = (P + KTC - 1) / KTC;
  // Key tile 0 is the suffix (this request's own <= 64 keys); key tile g >= 1 is prefix keys [(g-1) * 64, g * 64).
  // Softmax does not care about the order.  With num_splits > 1 (grids far below one wave: few requests) the CTA takes
  // key tiles [g_lo, g_lo + T) of the Tp + 1 and leaves its unnormalised result for the merge kernel.
  const int ns = a.num_splits > 1 ? a.num_splits : 1, split = blockIdx.z;
  const int g_lo = (int)(((long long)(Tp + 1) * split) / ns);
  const int T = (int)(((long long)(Tp + 1) * (split + 1)) / ns) - g_lo;
  if (T <= 0) {
    // a request with fewer key tiles than splits: this range is empty, the merge kernel skips it
    if (tid >= 160) {
      const int row = tid - 160, hl = row >> 6, i = row & 63;
      if (i < S) {
        const size_t slab = ((size_t)(b * d.Hq + head0 + hl) * ns + split) * QROWS + i;
        a.part_ml[slab * 2] = -INFINITY, a.part_ml[slab * 2 + 1] = 0.f;
      }
    }
    __syncthreads();
    if (warp == 4) {
      tc_fence_after();
      tmem_dealloc(tmem_base, COLS);
    }
    return;
  }

  // ---- loader state (warps 0-3): warps 0-1 stream K tiles, warps 2-3 stream V tiles -----------------
  const bool is_v = warp >= 2;
  const int lt2 = tid & 63;                  // thread within its stream
  const int lc = lt2 & 31, r0 = lt2 >> 5;    // 16-byte chunk column; rows r0, r0 + 2, ...
  const size_t kv_stride = (size_t)d.Hkv * DH * 2;
  const uint8_t* G = reinterpret_cast<const uint8_t*>(r.prefix_kv) +
                     (((size_t)(a.layer * 2 + (is_v ? 1 : 0)) * r.kv_tokens + p0) * d.Hkv + hk) * (DH * 2) + (size_t)lc * 16;
  const uint32_t tile_base = (is_v ? Vs : Ks) + (uint32_t)(lc >> 3) * KV_BLOCK;
  auto issue = [&](int t) {                  // local tile t of a prefix key tile (g_lo + t >= 1)
    const int gt = g_lo + t;
    const uint32_t tb = tile_base + (uint32_t)(t % NKV) * KV_BYTES;
    const int rows = min(KTC, P - (gt - 1) * KTC);
    const uint8_t* g0 = G + (size_t)(gt - 1) * KTC * kv_stride;
#pragma unroll 8
    for (int row = r0; row < KTC; row += 2) {
      const bool ok = row < rows;            // rows past the prefix are zero-filled
      cp_async16(tb + (uint32_t)row * 128 + (uint32_t)(((lc & 7) ^ (row & 7)) << 4), g0 + (size_t)(ok ? row : 0) * kv_stride,
                 ok ? 16u : 0u);
    }
    cp_async_commit();
  };
  // ---- no CTA-wide prologue barrier: each stream publishes its own first tile, so S(0) starts as soon as Q and
  // the suffix keys are in place while the suffix values and the first prefix tiles are still in flight ----
  if (warp < 4) {
    // =========================== loaders ==========================================================
    // K buffer (t % 3) is free again once the logits of tile t exist (s_full), V buffer once P V of tile t has
    // completed (pv_done).  Tile t + 1 is published only after that wait: its consumer could not start
    // earlier anyway, and it keeps the waited barrier from running a whole phase ahead of the parity wait.
    uint64_t* full = is_v ? v_full : k_full;
    {
      if (g_lo == 0) {
        // key tile 0 = this request's own keys / values (rotated bf16 from the QKV epilogue); rows >= S are zero-filled
        const uint8_t* src = reinterpret_cast<const uint8_t*>(is_v ? a.vr : a.kr) + ((size_t)(b * d.Hkv + hk) * S) * (DH * 2) +
                             (size_t)lc * 16;
#pragma unroll 8
        for (int row = r0; row < KTC; row += 2) {
          const bool ok = row < S;
          cp_async16(tile_base + (uint32_t)row * 128 + (uint32_t)(((lc & 7) ^ (row & 7)) << 4),
                     src + (size_t)(ok ? row : 0) * (DH * 2), ok ? 16u : 0u);
        }
        cp_async_commit();
      } else {
        issue(0);
      }
      // The prefix tiles are requested only after tile 0 has landed: every CTA of the grid starts at the same time,
      // and requests issued together share the SM's ingest bandwidth, which would delay the data needed first.
      cp_async_wait<0>();
      fence_async_smem();
      if (is_v) group_sync<BAR_LOAD + 2, 64>(); else group_sync<BAR_LOAD, 64>();
      if (lt2 == 0) mbar_arrive_local(smem_u32(&full[0]));
      // (V buffers 1 and 2 are the staging area of the Q rows until the softmax warps have moved them to tensor memory)
      if (is_v) asm volatile("bar.sync %0, %1;" ::"n"(BAR_QSTAGE), "n"(192) : "memory");
      if (T > 1) issue(1);
      if (T > 2) issue(2);
    }
    for (int t = 0; t + 1 < T; ++t) {
      if (is_v) mbar_wait(smem_u32(&pv_done[t & 1]), (uint32_t)(t >> 1) & 1u, wc);
      else mbar_wait(smem_u32(&s_full[t & 1]), (uint32_t)(t >> 1) & 1u, wc);
      if (t + 2 < T) cp_async_wait<1>(); else cp_async_wait<0>();   // tile t + 1 has landed (t + 2 may be in flight)
      fence_async_smem();                    // generic-proxy writes, read next by the tensor core
      if (is_v) group_sync<BAR_LOAD + 2, 64>(); else group_sync<BAR_LOAD, 64>();
      if (lt2 == 0) mbar_arrive_local(smem_u32(&full[(t + 1) % NKV]));
      if (t + 3 < T) issue(t + 3);           // into the buffer tile t has just released
    }
  } else if (warp == 4) {
    // =========================== MMA issuer ========================================================
    // Order: S(0), S(1); then for every tile t: P(t) V(t), S(t+2).  With two S buffers in TMEM the logits are
    // always ready one tile before the softmax warps want them.
    auto issue_s = [&](int t) {
      const int buf = t & 1, kbuf = t % NKV;
      // (S buffer `buf` last held P of tile t - 2, whose P V was issued before this: the tensor pipe runs in order)
      const bool ok = mbar_wait(smem_u32(&k_full[kbuf]), (uint32_t)(t / NKV) & 1u, wc);
      tc_fence_after();
      const uint32_t kb = Ks + (uint32_t)kbuf * KV_BYTES;
      if (__all_sync(0xffffffffu, ok)) {
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {
          const uint64_t db = make_desc(kb + (uint32_t)(kk >> 2) * KV_BLOCK + (uint32_t)(kk & 3) * 32);
          if (elect_one()) umma_bf16_ts(tmem_s + (uint32_t)buf * KTC, tmem_q + (uint32_t)kk * 8, db, IDESC_S, kk > 0 ? 1u : 0u);
        }
      }
      if (elect_one()) umma_commit(smem_u32(&s_full[buf]));
      __syncwarp();
    };
    {
      mbar_wait(smem_u32(&q_full), 0u, wc);    // Q is in tensor memory
      tc_fence_after();
      if (lane == 0) trace_stamp(trc, 2);
    }
    issue_s(0);
    if (lane == 0) trace_stamp(trc, 3);
    if (T > 1) issue_s(1);
    for (int t = 0; t < T; ++t) {
      const int buf = t & 1, vbuf = t % NKV;
      const uint32_t vb = Vs + (uint32_t)vbuf * KV_BYTES;
      bool ok = mbar_wait(smem_u32(&v_full[vbuf]), (uint32_t)(t / NKV) & 1u, wc);
      ok = mbar_wait(smem_u32(&p_full[buf]), (uint32_t)(t >> 1) & 1u, wc) && ok;
      tc_fence_after();
      if (__all_sync(0xffffffffu, ok)) {
#pragma unroll
        for (int kj = 0; kj < KTC / 16; ++kj) {
          // A = P of this tile: bf16 pairs in the first 32 columns of S buffer `buf`
          const uint64_t db = make_desc_mn(vb + (uint32_t)kj * (16 * 128), KV_BLOCK, 1024);
          if (elect_one())
            umma_bf16_ts(tmem_o, tmem_s + (uint32_t)buf * KTC + (uint32_t)kj * 8, db, IDESC_PV, (t > 0 || kj > 0) ? 1u : 0u);
        }
      }
      if (elect_one()) umma_commit(smem_u32(&pv_done[buf]));
      __syncwarp();
      if (t + 2 < T) issue_s(t + 2);
      if (t == 0 && lane == 0) trace_stamp(trc, 4);
    }
    if (lane == 0) trace_stamp(trc, 5);
    if (*reinterpret_cast<volatile int*>(&abort_flag)) {
      // a wait was given up: the softmax warps no longer wait for the tensor core, so make sure here that every MMA
      // issued above has completed before tensor memory is released below
      if (elect_one()) umma_commit(smem_u32(&fin_bar));
      __syncwarp();
      for (uint32_t it = 0; it < DRAIN_LIMIT && !mbar_test(smem_u32(&fin_bar), 0u); ++it) __nanosleep(64);
    }
  } else {
    // =========================== softmax / correction / output =====================================
    const int st = tid - 160;                 // 0..127
    const int q = warp & 3;
    const int row = q * 32 + lane;            // accumulator row = TMEM lane
    const int hl = row >> 6, i = row & 63;
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    float m = -INFINITY, l = 0.f;             // running maximum (log2 units) and sum
    {
      // Q (already rotated, scaled bf16) -> tensor memory, where it is the A operand of every S = Q K^T (two bf16 per
      // 32-bit column, in memory order), one row per thread.  A row is 2 DH bytes of global memory: read by its own
      // thread, one 16-byte load would touch 32 different lines per warp instruction.  Each warp instead copies its 32
      // rows (contiguous in global memory) with coalesced 16-byte cp.async into a staging block (V buffers 1 and 2,
      // not needed before the second key tile's P V; 16-byte chunks XOR-swizzled by the row so that both the row-wise
      // writes and the one-row-per-thread reads are free of bank conflicts), and every thread then reads its row.
      constexpr int QROW = DH * 2;                                  // bytes per row
      constexpr int QCH = QROW / 16;                                // 16-byte chunks per row (32)
      static_assert(4 * 32 * QROW <= 2 * KV_BYTES, "Q staging exceeds two V buffers");
      const uint32_t qstage = Vs + KV_BYTES + (uint32_t)q * (32 * QROW);
      const int i0 = (q * 32) & 63;                                 // first token of this warp's 32 rows
      const uint8_t* qsrc = reinterpret_cast<const uint8_t*>(a.qr + ((size_t)(b * d.Hq + head0 + hl) * S) * DH);
#pragma unroll 8
      for (int rr = 0; rr < 32; ++rr) {
        const bool ok = i0 + rr < S;                                // rows past the suffix are zero-filled
        for (int c = lane; c < QCH; c += 32)
          cp_async16(qstage + (uint32_t)rr * QROW + (uint32_t)((c ^ (rr & (QCH - 1))) << 4),
                     qsrc + (size_t)(ok ? i0 + rr : 0) * QROW + (size_t)c * 16, ok ? 16u : 0u);
      }
      cp_async_commit();
      cp_async_wait<0>();
      __syncwarp();
      const uint32_t qrow = qstage + (uint32_t)lane * QROW;
      const uint32_t qdst = tmem_q + lane_addr;
#pragma unroll 1
      for (int c = 0; c < DH / 2; c += 64) {                      // 64 columns = 128 bf16 = 16 x 16 bytes per round
        uint4 v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          const int ch = (c >> 2) + u;
          asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(v[u].x), "=r"(v[u].y), "=r"(v[u].z), "=r"(v[u].w)
                       : "r"(qrow + (uint32_t)((ch ^ (lane & (QCH - 1))) << 4))
                       : "memory");
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) tmem_st16u(qdst + (uint32_t)(c + 16 * u), reinterpret_cast<const uint32_t*>(v + 4 * u));
      }
      // the staging area goes back to the V loaders
      asm volatile("bar.arrive %0, %1;" ::"n"(BAR_QSTAGE), "n"(192) : "memory");
      tmem_st_wait();
      tc_fence_before();
      group_sync<BAR_SOFT, 128>();
      if (st == 0) mbar_arrive_local(smem_u32(&q_full));
    }
    const bool causal_row = d.block_causal && d.ns && i == 0;
    for (int t = 0; t < T; ++t) {
      mbar_wait(smem_u32(&s_full[t & 1]), (uint32_t)(t >> 1) & 1u, wc);
      tc_fence_after();
      const int gt = g_lo + t;
      const int valid = gt == 0 ? S : min(KTC, P - (gt - 1) * KTC);
      float s[KTC];
      tmem_ld64(tmem_s + (uint32_t)(t & 1) * KTC + lane_addr, s);
      if (valid < KTC) {
#pragma unroll
        for (int c = 0; c < KTC; ++c) s[c] = c < valid ? s[c] : -INFINITY;
      }
      if (causal_row && gt == 0) {            // the state token sees, of the suffix, only itself
#pragma unroll
        for (int c = 1; c < KTC; ++c) s[c] = -INFINITY;
      }
      float mx = s[0];
#pragma unroll
      for (int c = 1; c < KTC; ++c) mx = fmaxf(mx, s[c]);
      mx *= LOG2E;
      // running maximum: keep the old one unless the new exceeds it by more than the threshold
      float m_new = m;
      if (mx > m + RESCALE_THRESHOLD || m == -INFINITY) m_new = fmaxf(m, mx);
      const bool rescale = m_new != m && m != -INFINITY;
      const float corr = rescale ? exp2f(m - m_new) : 1.0f;
      const float nsub = m_new == -INFINITY ? 0.f : -m_new;
      float rs = 0.f;
      // P overwrites this thread's own row of the S buffer it has just read (bf16 pairs, first 32 columns):
      // it is the A operand of P V, read from tensor memory
      const uint32_t pdst = tmem_s + (uint32_t)(t & 1) * KTC + lane_addr;
#pragma unroll
      for (int c16 = 0; c16 < KTC / 32; ++c16) {
        uint32_t w[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float e0 = ex2_fast(fmaf(s[c16 * 32 + 2 * e], LOG2E, nsub)), e1 = ex2_fast(fmaf(s[c16 * 32 + 2 * e + 1], LOG2E, nsub));
          rs += e0 + e1;
          w[e] = pack_bf16(e0, e1);
        }
        tmem_st16u(pdst + (uint32_t)c16 * 16, w);
      }
      l = l * corr + rs;
      m = m_new;
      if (__any_sync(0xffffffffu, rescale)) {     // rare: rescale this warp's 32 accumulator rows
        // every P V issued so far must have completed before O is touched
        mbar_wait(smem_u32(&pv_done[(t - 1) & 1]), (uint32_t)((t - 1) >> 1) & 1u, wc);
        tc_fence_after();
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
      tmem_st_wait();
      tc_fence_before();
      group_sync<BAR_SOFT, 128>();
      if (st == 0) mbar_arrive_local(smem_u32(&p_full[t & 1]));
    }
    // ---- output: O / l -> bf16 ----
    const bool okf =
        __all_sync(0xffffffffu, mbar_wait(smem_u32(&pv_done[(T - 1) & 1]), (uint32_t)((T - 1) >> 1) & 1u, wc));
    tc_fence_after();
    if (st == 0) trace_stamp(trc, 6);
    if (ns > 1) {
      // Split key range: the unnormalised accumulator rows (fp32) and (running maximum in log2 units, sum) of this
      // range go to the merge kernel.  A row is 4 DH bytes of global memory: staged per warp (64 columns = 256 bytes
      // per row at a time, 16-byte chunks XOR-swizzled by the row) and copied out with coalesced 16-byte stores.
      const int i0 = (q * 32) & 63;
      const int nrow = okf ? max(0, min(32, S - i0)) : 0;
      const size_t slab = ((size_t)(b * d.Hq + head0 + hl) * ns + split) * QROWS + i0;   // first row of this warp
      if (lane < nrow) {
        a.part_ml[(slab + lane) * 2] = m;
        a.part_ml[(slab + lane) * 2 + 1] = l;
      }
      const uint32_t ostage = Ks + (uint32_t)q * 8192u;
#pragma unroll 1
      for (int c = 0; c < DH; c += 64) {
        float o[64];
        tmem_ld64(tmem_o + lane_addr + (uint32_t)c, o);
#pragma unroll
        for (int e = 0; e < 64; e += 4)
          asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(ostage + (uint32_t)lane * 256u + (uint32_t)((((e >> 2) ^ (lane & 15))) << 4)),
                       "f"(o[e]), "f"(o[e + 1]), "f"(o[e + 2]), "f"(o[e + 3])
                       : "memory");
        __syncwarp();
        for (int idx = lane; idx < nrow * 16; idx += 32) {
          const int rr = idx >> 4, ch = idx & 15;
          float4 v;
          asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                       : "r"(ostage + (uint32_t)rr * 256u + (uint32_t)((ch ^ (rr & 15)) << 4)) : "memory");
          *reinterpret_cast<float4*>(a.part_o + (slab + rr) * DH + c + ch * 4) = v;
        }
        __syncwarp();
      }
    } else if (a.rows_pad > 0) {
      // O / l -> bf16 in the tiled layout of the O projection's input.  A thread holds one row; its 128 bytes of a
      // 64-channel k-chunk go to a staging block of the warp (the K buffers are free: every MMA has completed) at the
      // position they have in global memory, where the warp's 32 rows of a k-chunk are one contiguous range, and the
      // warp then copies that range with coalesced 16-byte stores (one row per thread, stored directly, would touch 32
      // lines per instruction).
      const float inv = 1.0f / l;
      const int i0 = (q * 32) & 63;
      const int orow = b * S + i0 + lane, head = head0 + hl;
      const int nrow = okf ? max(0, min(32, S - i0)) : 0;        // rows of this warp that exist
      const uint32_t ostage = Ks + (uint32_t)q * 4096u;
      const uint32_t orow_s = ostage + (uint32_t)lane * 128u;
#pragma unroll 1
      for (int c = 0; c < DH; c += 64) {
        float o[64];
        tmem_ld64(tmem_o + lane_addr + (uint32_t)c, o);         // four loads in flight, one wait
#pragma unroll
        for (int e = 0; e < 64; e += 8) {
          const uint32_t w0 = pack_bf16(o[e] * inv, o[e + 1] * inv), w1 = pack_bf16(o[e + 2] * inv, o[e + 3] * inv);
          const uint32_t w2 = pack_bf16(o[e + 4] * inv, o[e + 5] * inv), w3 = pack_bf16(o[e + 6] * inv, o[e + 7] * inv);
          asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(orow_s + (uint32_t)((((e >> 3) ^ (orow & 7))) << 4)), "r"(w0),
                       "r"(w1), "r"(w2), "r"(w3)
                       : "memory");
        }
        __syncwarp();
        // k-chunk (head * DH + c) / 64 of the output, rows b * S + i0 ..: nrow * 128 contiguous bytes
        uint4* dst = reinterpret_cast<uint4*>(a.out + ((size_t)((head * DH + c) >> 6) * a.rows_pad + (size_t)(b * S + i0)) * 64);
        for (int idx = lane; idx < nrow * 8; idx += 32) {
          uint4 v;
          asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(ostage + (uint32_t)idx * 16u) : "memory");
          dst[idx] = v;
        }
        __syncwarp();
      }
    } else {
      const bool wr = okf && i < S;             // the TMEM loads stay warp-uniform; only the stores are predicated
      const float inv = 1.0f / l;
      const int orow = b * S + (i < S ? i : 0), head = head0 + hl;
#pragma unroll 1
      for (int c = 0; c < DH; c += 64) {
        float o[64];
        tmem_ld64(tmem_o + lane_addr + (uint32_t)c, o);         // four loads in flight, one wait
#pragma unroll
        for (int e = 0; e < 64; e += 8) {
          const uint4 w = make_uint4(pack_bf16(o[e] * inv, o[e + 1] * inv), pack_bf16(o[e + 2] * inv, o[e + 3] * inv),
                                     pack_bf16(o[e + 4] * inv, o[e + 5] * inv), pack_bf16(o[e + 6] * inv, o[e + 7] * inv));
          if (wr) *reinterpret_cast<uint4*>(a.out + out_index(orow, head * DH + c + e, a.rows_pad, d.Nq)) = w;
        }
      }
    }
    tc_fence_before();
    if (st == 0 && trc) {
      unsigned long long tt_;
      unsigned sm;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(tt_)::"memory");
      asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
      trc[8] = tt_, trc[7] = sm, trc[9] = (unsigned long long)T, trc[10] = 1;   // ([10]: marks an attention slot)
    }
  }

  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem_base, COLS);
  }
}

template <int DH>
constexpr size_t attn_tc_smem() {
  return 1024 + 2 * (size_t)NKV * KTC * DH * 2;
}

}  // namespace

// Key-range splits of the tcgen05 attention kernel: only for grids far below one wave (few requests), at most 8 and
// at most the key tiles of the longest prefix (a request with fewer key tiles leaves some of its ranges empty).
int attention_tc_splits(const Dims& d, int batch, int n_sm, int max_prefix) {
  const int ctas = batch * (d.Hq / 2);
  int want = n_sm / (ctas > 0 ? ctas : 1);
  const int tiles = (max_prefix + KTC - 1) / KTC + 1;
  if (want > tiles) want = tiles;
  if (want > 8) want = 8;
  // (measured on the pi0-shaped expert, 816-token prefixes: 4 requests 12.2 -> 11.3 ms per call with 8 ranges,
  // 8 requests 12.9 -> 12.6 ms with 4, 16 requests 16.8 -> 17.6 ms with 2: the merge kernel and the fp32 partials cost
  // more than two ranges save)
  return want < 4 ? 1 : want;
}

bool attention_tc_supported(const Dims& d) {
  return d.dh == 256 && d.S <= 64 && d.Hq % 2 == 0 && (d.Hq / d.Hkv) % 2 == 0;
}

cudaError_t launch_attention_tc(const Request* rq, int* status, const __nv_bfloat16* qr, const __nv_bfloat16* kr,
                                const __nv_bfloat16* vr, int layer, __nv_bfloat16* out_tiled, int rows_pad, const Dims& d,
                                int batch, const int* order, unsigned wait_limit, cudaStream_t st, unsigned long long* trace,
                                int num_splits, float* scratch) {
  static PerDeviceOnce once;
  if (once.needed()) {
    cudaError_t e = cudaFuncSetAttribute(k_attn_tc<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)attn_tc_smem<256>());
    if (e != cudaSuccess) return e;
    once.done();
  }
  AttnArgs a{};
  a.rq = rq, a.status = status, a.qr = qr, a.kr = kr, a.vr = vr, a.layer = layer, a.out = out_tiled, a.rows_pad = rows_pad;
  if (num_splits > 1 && !scratch) return cudaErrorInvalidValue;
  a.num_splits = num_splits > 1 ? num_splits : 1, a.d = d, a.wait_limit = wait_limit, a.order = order, a.trace = trace;
  a.part_o = scratch;
  a.part_ml = scratch ? scratch + (size_t)batch * d.Hq * a.num_splits * QROWS * d.dh : nullptr;
  dim3 grid(d.Hq / 2, batch, a.num_splits);
  cudaError_t e = launch_pdl(k_attn_tc<256>, grid, dim3(288), attn_tc_smem<256>(), st, a);
  if (e == cudaSuccess && a.num_splits > 1)
    e = launch_attention_merge(status, a.part_o, a.part_ml, out_tiled, rows_pad, a.num_splits, d, batch, st);
  return e;
}

}  // namespace phyai
