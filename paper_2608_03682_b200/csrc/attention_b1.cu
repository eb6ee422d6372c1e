// Suffix -> (prefix U suffix) attention for calls with very few requests (batch 1): tcgen05 tensor cores, the key
// range of a request split over a thread-block cluster, partial results merged over distributed shared memory.
//
// Work split.  Few queries, one long shared K / V stream: the limiter is how fast the prefix K / V (and Q) get into
// the SMs, so the keys of a request are divided among the 8 CTAs of a cluster (an eighth of the prefix keys plus an
// eighth of the request's own suffix keys each, <= 128 keys: ONE 128-key tile per CTA for prefixes up to ~970 tokens,
// hence no online-softmax loop in the common case).  A CTA takes HPC query heads: one (rows 0..63 of the 128-row MMA;
// the Q tile, the partials that cross the cluster and the merge are then half as large, and the call runs on 8 Hq
// CTAs) or, when the SMs do not allow that many CTAs, two heads that share a kv head stacked on the M axis.
// Grid = (8 key ranges, Hq / HPC, requests).
//   S = Q K^T   tcgen05.mma M = 128, N = 128 keys, K = head_dim; Q and the K tile in shared memory
//   softmax     one thread per row straight from tensor memory (no shuffles); P (bf16) written back to tensor memory
//   O = P V     tcgen05.mma M = 128, N = head_dim, K = 128 keys; P is the tensor-memory A operand, V an MN-major B
//               operand (K and V tiles share one shared-memory layout and loader code)
// The prefix rows of a CTA's tile are constants of the call and are requested before the programmatic dependency
// wait; Q (written by the QKV projection's epilogue as this kernel's swizzled operand tile: eight bulk copies) and the
// CTA's share of the request's own (suffix) keys come right after it.
//
// Merge.  Every CTA holds an un-normalised partial (O, row max, row sum) of all HPC x S rows.  Row i of every head is
// owned by CTA i / 8: each CTA writes its partial, rounded to bf16 and grouped by owner, into its own shared memory
// and sends every owner one bulk copy over distributed shared memory (counted on the owner's mbarrier); the owner
// combines the 8 partials of its rows in rank order and stores the normalised bf16 rows as the activation tile of
// the output projection.  No partials in global memory, no merge kernel.
//
// Warps: 4 issues the MMAs; the other eight are two threads per accumulator row (each half of the columns): the
// softmax, partial out; warps 0-1 also load K, 2-3 V (16-byte cp.async into the swizzled block
// layout); all nine merge.  Waits are bounded (see mbar_wait_drain); after a give-up the
// protocol still runs to its end so that no peer is left waiting, only the global stores are skipped.
#include "attention.cuh"
#include "tc.cuh"

namespace phyai {
namespace {

constexpr int KB = 128;            // keys per tile
// Named barriers: the eight row warps among themselves; row warps -> MMA warp "operands of the tile are in shared
// memory" and "P is in tensor memory" (the 256 row threads arrive without waiting, the MMA warp waits: a hardware
// wake-up instead of a polled mbarrier, which measured 0.75 us from arrival to the MMA warp's next instruction).
constexpr int BAR_ROWS = 1, BAR_QK = 2, BAR_P = 3;
template <int BAR, int NT>
__device__ __forceinline__ void named_arrive() {
  asm volatile("bar.arrive %0, %1;" ::"n"(BAR), "n"(NT) : "memory");
}

template <int DH, int HPC>
struct B1Layout {
  static constexpr int BLOCK = KB * 128;                     // one 64-channel block of a K / V tile: 128 keys x 128 bytes
  static constexpr int TILE = (DH / 64) * BLOCK;             // a K or V tile
  static constexpr int PITCH = DH * 2 + 16;                  // bf16 partial row, padded against bank conflicts
  static constexpr int SLOT = HPC * 8 * (PITCH + 16);        // one owner's block: HPC heads x 8 rows of O, then their (max, sum)
                                                             // in 16-byte entries (a bulk copy moves multiples of 16 bytes)
  static constexpr int QTILE = 128 * DH * 2;                 // the Q operand (128 rows; with one head the upper 64 idle)
  static constexpr int RECV = 8 * SLOT > QTILE ? 8 * SLOT : QTILE;   // receive area of the merge; first holds Q
  static constexpr size_t SMEM = 1024 + 2 * (size_t)TILE + (size_t)RECV;
};

template <int DH, int HPC>
__global__ void __launch_bounds__(288, 1) k_attn_b1(const AttnArgs a) {
  using L = B1Layout<DH, HPC>;
  constexpr int COLS = 512;                   // S / P at columns [0, 128), O at [128, 128 + DH)
  constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(KB >> 3) << 17) | ((128u >> 4) << 24);
  constexpr uint32_t IDESC_PV =
      (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((128u >> 4) << 24);

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t s_full, pv_done, mrg_bar, q_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag, suppress, mrg_ok;
  __shared__ float wtab[16][8];               // merge: weight of partial s for each of my (up to 2 x 8) rows
  __shared__ float xch[2][128], xsum[2][128]; // softmax: the two half-row threads exchange their maximum and sum

  const Dims& d = a.d;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rank = blockIdx.x, hp = blockIdx.y, b = blockIdx.z;
  const int head0 = hp * HPC;
  const int hk = head0 / (d.Hq / d.Hkv);
  const int S = d.S;                                      // query rows per head
  const int Sk = d.Sk > 0 ? d.Sk : d.S;                   // the request's own (suffix) keys that exist ...
  const int Sk_stride = d.Sk_stride > 0 ? d.Sk_stride : d.S;   // ... and their row pitch per kv head
  // tracing: one CTA of the launch, or (trace_all) every CTA into the slot of its linear index
  const bool tcta = a.trace && (a.trace_all || (rank == 0 && hp == 0 && b == 0));
  unsigned long long* const trp = a.trace_all ? a.trace + (size_t)((b * gridDim.y + hp) * gridDim.x + rank) * 16 : a.trace;
  const bool tracer = tid == 0 && tcta;

  pdl_launch_dependents();
  if (tracer) trace_stamp(trp, 0);
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t Ks = base, Vs = base + L::TILE;
  const uint32_t stg = base;                              // partial, grouped by owner: over the K / V tiles once they are dead
  const uint32_t recv = base + 2 * L::TILE;               // [8 sources][SLOT]
  const uint32_t Qs = recv;                               // Q tile (2 heads x 64 rows), until the logits exist
  const int n_me = max(0, min(8, S - rank * 8));          // suffix rows (per head) this CTA owns in the merge
  const uint32_t my_bytes = (uint32_t)(HPC * n_me * (L::PITCH + 16));

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&s_full), 1), mbar_init(smem_u32(&pv_done), 1);
    mbar_init(smem_u32(&mrg_bar), 1);
    mbar_init(smem_u32(&q_bar), 8);
    if (n_me > 0) mbar_expect_tx(smem_u32(&mrg_bar), 7u * my_bytes);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    tmem_alloc(smem_u32(&tmem_slot), COLS);
    tc_fence_before();
  }
  // every CTA's barriers exist before a peer can send to them (this is before the dependency wait)
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + KB;
  const WaitCtx wc{a.status, &abort_flag, a.wait_limit};

  // (the request block is written before the captured loop starts: safe to read ahead of the dependency wait)
  const Request r = *a.rq;
  const int p0 = r.cu_lens[b], P = r.cu_lens[b + 1] - p0;
  // Keys of this CTA: an eighth of the prefix keys followed by an eighth of the request's own (suffix) keys -- the
  // suffix rows only exist after the dependency wait, so every CTA fetches its share of them then, not one CTA all.
  const int pre_lo = (int)(((long long)P * rank) / 8), n_pre = (int)(((long long)P * (rank + 1)) / 8) - pre_lo;
  const int suf_lo = (Sk * rank) / 8, n_suf = (Sk * (rank + 1)) / 8 - suf_lo;
  const int n_keys = n_pre + n_suf;
  const int T = (n_keys + KB - 1) / KB;                   // tiles of this CTA (1 unless P + S > 1024; 0 for an empty range)

  if (warp == 4) {
    // =========================== MMA issuer ======================================================================
    pdl_wait();
    // (this warp never touches the receive area: its part in the cluster barrier that guards it, see the row warps)
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    if (lane == 0) suppress = status_set(a.status) ? 1 : 0;
    for (int t = 0; t < T; ++t) {
      const bool trm = lane == 0 && tcta && t == 0;
      group_sync<BAR_QK, 288>();              // the K / V tile is in shared memory
      if (t == 0) mbar_wait_drain(smem_u32(&q_bar), 0u, wc);    // ... and the Q tile (one bulk copy)
      tc_fence_after();
      if (trm) trace_stamp(trp, 14);
#pragma unroll
      for (int kk = 0; kk < DH / 16; ++kk) {
        const uint64_t db = make_desc(Ks + (uint32_t)(kk >> 2) * L::BLOCK + (uint32_t)(kk & 3) * 32);
        const uint64_t da = make_desc(Qs + (uint32_t)(kk >> 2) * L::BLOCK + (uint32_t)(kk & 3) * 32);
        if (elect_one()) umma_bf16(tmem_s, da, db, IDESC_S, kk > 0 ? 1u : 0u);
      }
      if (elect_one()) umma_commit(smem_u32(&s_full));
      __syncwarp();
      if (trm) trace_stamp(trp, 15);
      group_sync<BAR_P, 288>();               // P is in tensor memory
      tc_fence_after();
#pragma unroll
      for (int kj = 0; kj < KB / 16; ++kj) {
        // A = P of this tile: bf16 pairs in the first 64 columns of the S buffer
        const uint64_t db = make_desc_mn(Vs + (uint32_t)kj * (16 * 128), L::BLOCK, 1024);
        if (elect_one()) umma_bf16_ts(tmem_o, tmem_s + (uint32_t)kj * 8, db, IDESC_PV, (t > 0 || kj > 0) ? 1u : 0u);
      }
      if (elect_one()) umma_commit(smem_u32(&pv_done));
      __syncwarp();
    }
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  } else {
    // =========================== the eight row warps ==============================================================
    // Two threads per accumulator row (same TMEM lane quarter = warp % 4): group 0 (warps 5-8) takes the first half of
    // a row's columns, group 1 (warps 0-3) the second half -- of Q on its way into tensor memory, of the logits in the
    // softmax, of O on its way out.  Group 1 also loads the tiles: warps 0-1 K, warps 2-3 V.
    const int g = warp < 4 ? 1 : 0;
    const int q = warp & 3;
    const int row = q * 32 + lane;            // accumulator row = TMEM lane
    const int hl = row >> 6, i = row & 63;
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    const bool lead = warp == 5 && lane == 0;
    const bool tr2 = lead && tcta;
    float m = -INFINITY, l = 0.f;             // running maximum (log2 units) and sum
    // ---- loader state (group 1) ----
    const bool is_v = warp >= 2;
    const int lt2 = tid & 63;
    constexpr int CHUNKS = DH / 8, RSTEP = 64 / CHUNKS;   // 16-byte chunks per row; rows covered by the 64 threads at once
    const int lc = lt2 % CHUNKS, r0 = lt2 / CHUNKS;       // 16-byte chunk column; rows r0, r0 + RSTEP, ...
    const size_t kv_stride = (size_t)d.Hkv * DH * 2;
    const uint8_t* Gp = reinterpret_cast<const uint8_t*>(r.prefix_kv) +
                        (((size_t)(a.layer * 2 + (is_v ? 1 : 0)) * r.kv_tokens + p0) * d.Hkv + hk) * (DH * 2) + (size_t)lc * 16;
    const uint8_t* Gs = reinterpret_cast<const uint8_t*>(is_v ? a.vr : a.kr) + ((size_t)(b * d.Hkv + hk) * Sk_stride) * (DH * 2) +
                        (size_t)lc * 16;
    const uint32_t tile_base = (is_v ? Vs : Ks) + (uint32_t)(lc >> 3) * L::BLOCK;
    // rows of tile t: the prefix rows when `prefix` is set, otherwise the request's own (suffix) rows and, for V, zeros
    // in the rows past the range (their probabilities are 0, but 0 x stale shared memory must stay 0; K rows past the
    // range only produce logits that the softmax masks).  The loops walk exactly the rows they copy.
    auto issue = [&](int t, bool prefix) {
      const int np = max(0, min(KB, n_pre - t * KB));        // prefix rows of the tile
      const int nv = max(0, min(KB, n_keys - t * KB));       // rows that exist
      if (prefix) {
        const uint8_t* src = Gp + (size_t)(pre_lo + t * KB + r0) * kv_stride;
        for (int row2 = r0; row2 < np; row2 += RSTEP, src += (size_t)RSTEP * kv_stride)
          cp_async16(tile_base + (uint32_t)row2 * 128 + (uint32_t)(((lc & 7) ^ (row2 & 7)) << 4), src, 16u);
      } else {
        for (int row2 = np + r0; row2 < nv; row2 += RSTEP)
          cp_async16(tile_base + (uint32_t)row2 * 128 + (uint32_t)(((lc & 7) ^ (row2 & 7)) << 4),
                     Gs + (size_t)(suf_lo + t * KB + row2 - n_pre) * (DH * 2), 16u);
        if (is_v)
          for (int row2 = nv + r0; row2 < KB; row2 += RSTEP)
            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(tile_base + (uint32_t)row2 * 128 + (uint32_t)(((lc & 7) ^ (row2 & 7)) << 4)),
                         "r"(0u)
                         : "memory");
      }
    };
    if (g == 1 && T > 0) issue(0, true);      // constants of the call: ahead of the dependency wait
    if (g == 1) cp_async_commit();
    pdl_wait();
    if (tr2) trace_stamp(trp, 1);
    if (T > 0) {
      if (g == 1) {
        issue(0, false);
        cp_async_commit();
      }
      // Q (rotated, scaled bf16) was written by the QKV projection as this kernel's operand tile: one bulk copy into the
      // receive area of the merge (idle until the peers push).  (16-byte asynchronous copies by all row threads took
      // 1.5 us for the 64 KB; one thread per row straight into tensor memory 3.3 us.)
      // (an eighth per row warp: the copies of one warp complete one after the other, those of different warps overlap)
      if (lane == 0) {
        constexpr uint32_t QBYTES = 128u * DH * 2u;
        const int part = warp < 4 ? warp : warp - 1;
        const uint8_t* qt = reinterpret_cast<const uint8_t*>(a.qr) + (size_t)(b * (d.Hq >> 1) + (head0 >> 1)) * QBYTES;
        if (HPC == 2) {
          constexpr uint32_t QPART = QBYTES / 8;
          mbar_expect_tx(smem_u32(&q_bar), QPART);
          bulk_g2s(Qs + (uint32_t)part * QPART, qt + (size_t)part * QPART, QPART, smem_u32(&q_bar));
        } else {
          // one head: its 64 rows of every 64-channel block of the pair's tile (the other 64 rows of the MMA idle)
          constexpr uint32_t PARTS = 8 / (DH / 64), QPART = 8192u / PARTS;      // pieces per block, bytes per piece
          const uint32_t kb = (uint32_t)part / PARTS, pc = (uint32_t)part % PARTS;
          mbar_expect_tx(smem_u32(&q_bar), QPART);
          bulk_g2s(Qs + kb * (uint32_t)L::BLOCK + pc * QPART, qt + (size_t)kb * L::BLOCK + (size_t)(head0 & 1) * 8192 + pc * QPART, QPART,
                   smem_u32(&q_bar));
        }
      }
      cp_async_wait<0>();                                          // (group 1: its tile rows as well)
      fence_async_smem();                                          // generic-proxy writes, read next by the tensor core
      if (tr2) trace_stamp(trp, 10);
      named_arrive<BAR_QK, 288>();
    }

    if (tr2) trace_stamp(trp, 2);
    const bool causal_row = d.block_causal && d.ns && i == 0;
    for (int t = 0; t < T; ++t) {
      const uint32_t ph = (uint32_t)t & 1u;
      if (t > 0) {
        // single K / V buffers: tile t may be fetched once P V of tile t - 1 has completed (rare: P + S > 1024)
        if (warp == 5) mbar_wait_drain(smem_u32(&pv_done), (uint32_t)(t - 1) & 1u, wc);
        group_sync<BAR_ROWS, 256>();
        if (g == 1) {
          issue(t, true);
          issue(t, false);
          cp_async_commit();
          cp_async_wait<0>();
          fence_async_smem();
        }
        named_arrive<BAR_QK, 288>();
      }
      // one warp polls the barrier, the other seven wait for it at the named barrier (in hardware): 256 polling threads
      // would share the shared-memory port with the operand reads of the MMAs they are waiting for
      if (warp == 5) mbar_wait_drain(smem_u32(&s_full), ph, wc);
      group_sync<BAR_ROWS, 256>();
      tc_fence_after();
      // (the last logits exist: the Q tile is dead and the receive area free -- see the cluster barrier ahead of the push)
      if (t == T - 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
      if (tr2) trace_stamp(trp, 11);
      // the visible key columns of this row form a prefix of the tile: the keys that exist, and for the state-token row
      // under the block-causal mask only the prefix keys and its own key (suffix key 0, in the first CTA's range)
      int nvis = min(KB, n_keys - t * KB);
      if (causal_row) nvis = min(nvis, max(0, n_pre + (suf_lo == 0 && n_suf > 0 ? 1 : 0) - t * KB));
      nvis -= g * 64;                         // relative to this thread's 64 columns
      float s[64];
      tmem_ld64(tmem_s + lane_addr + (uint32_t)(g * 64), s);
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int c = 0; c < 64; ++c) {
        s[c] = c < nvis ? s[c] : -INFINITY;
        mx4[c & 3] = fmaxf(mx4[c & 3], s[c]);
      }
      xch[g][row] = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      group_sync<BAR_ROWS, 256>();            // (also: both halves of every S row have been read -> P may overwrite them)
      const float mx = fmaxf(xch[0][row], xch[1][row]) * LOG2E;
      const float m_new = fmaxf(m, mx);
      const float corr = (m == -INFINITY) ? 1.0f : exp2f(m - m_new);
      const float nsub = m_new == -INFINITY ? 0.f : -m_new;
      // P = exp2(S log2e - m) as bf16 pairs over the first 64 columns of the S buffer (masked columns: exp2(-inf) = 0)
      float rs4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c16 = 0; c16 < 2; ++c16) {
        uint32_t w[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const int c = c16 * 32 + 2 * e;
          const float e0 = ex2_fast(fmaf(s[c], LOG2E, nsub)), e1 = ex2_fast(fmaf(s[c + 1], LOG2E, nsub));
          rs4[e & 3] += e0 + e1;
          w[e] = pack_bf16(e0, e1);
        }
        tmem_st16u(tmem_s + lane_addr + (uint32_t)(g * 32 + c16 * 16), w);
      }
      xsum[g][row] = (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
      if (t > 0) {
        // (rare path) the accumulator holds tiles 0..t-1 relative to the old maximum; P V of tile t - 1 has completed
        // (the tensor pipe runs in order and S of this tile was issued after it); each thread rescales its half row
#pragma unroll 1
        for (int c = g * (DH / 2); c < (g + 1) * (DH / 2); c += 16) {
          float o[16];
          tmem_ld16(tmem_o + lane_addr + (uint32_t)c, o);
#pragma unroll
          for (int e = 0; e < 16; ++e) o[e] *= corr;
          tmem_st16(tmem_o + lane_addr + (uint32_t)c, o);
        }
      }
      tmem_st_wait();
      tc_fence_before();
      named_arrive<BAR_P, 288>();
      group_sync<BAR_ROWS, 256>();            // (the other half row's sum is visible)
      l = l * corr + (xsum[0][row] + xsum[1][row]);
      m = m_new;
      if (tr2) trace_stamp(trp, 7);
    }
    if (T == 0) {
      if (g == 1) cp_async_wait<0>();
      asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    }
    // ---- partial out: half an O row -> bf16 into the owner's block of the staging area; group 0 adds (max, sum) ------
    if (T > 0 && warp == 5) mbar_wait_drain(smem_u32(&pv_done), (uint32_t)(T - 1) & 1u, wc);
    group_sync<BAR_ROWS, 256>();
    tc_fence_after();
    if (tr2) trace_stamp(trp, 3);
    {
      const int c = i >> 3, il = i & 7, n_c = max(0, min(8, S - c * 8));
      const bool wr = hl < HPC && i < S;
      const uint32_t blk = stg + (uint32_t)c * L::SLOT;
      const uint32_t rowp = blk + (uint32_t)(hl * n_c + il) * L::PITCH;
#pragma unroll 1
      for (int c0 = g * (DH / 2); c0 < (g + 1) * (DH / 2); c0 += 64) {
        float o[64];
        if (T > 0) {
          tmem_ld64(tmem_o + lane_addr + (uint32_t)c0, o);
        } else {
#pragma unroll
          for (int e = 0; e < 64; ++e) o[e] = 0.f;
        }
        if (wr) {
#pragma unroll
          for (int e = 0; e < 64; e += 8)
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(rowp + (uint32_t)(c0 + e) * 2), "r"(pack_bf16(o[e], o[e + 1])),
                         "r"(pack_bf16(o[e + 2], o[e + 3])), "r"(pack_bf16(o[e + 4], o[e + 5])), "r"(pack_bf16(o[e + 6], o[e + 7]))
                         : "memory");
        }
      }
      if (wr && g == 0)
        asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(blk + (uint32_t)(HPC * n_c) * L::PITCH + (uint32_t)(hl * n_c + il) * 16),
                     "f"(m), "f"(l)
                     : "memory");
    }
    tc_fence_before();
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the bulk-copy engine
    if (tr2) trace_stamp(trp, 12);
    group_sync<BAR_ROWS, 256>();
    // ---- every owner gets its block of my partial: one bulk copy over distributed shared memory -------------------
    // (first: every peer has moved its Q out of its receive area; all of them arrived long ago)
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    // (one copy per warp: the bulk copies issued by one warp complete one after the other)
    const int peer = warp < 4 ? warp : warp - 1;
    if (lane == 0 && peer != rank) {
      const int n_c = max(0, min(8, S - peer * 8));
      if (n_c > 0) {
        uint32_t dst, bar;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"(recv + (uint32_t)rank * L::SLOT), "r"(peer));
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar) : "r"(smem_u32(&mrg_bar)), "r"(peer));
        asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                     "r"(stg + (uint32_t)peer * L::SLOT), "r"((uint32_t)(HPC * n_c * (L::PITCH + 16))), "r"(bar)
                     : "memory");
      }
    }
    if (warp == 5) {
      bool ok = true;
      if (n_me > 0) ok = mbar_wait_drain(smem_u32(&mrg_bar), 0u, wc) > 0;
      if (lane == 0) mrg_ok = ok ? 1 : 0;
    }
  }
  __syncthreads();
  // From here on this CTA no longer needs its peers (what they sent has landed); it may leave once every peer says the
  // same, i.e. once every copy out of its own staging area has completed.  Arriving now and waiting at the very end
  // hides the skew between the CTAs behind the merge.
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  if (tracer) trace_stamp(trp, 4);

  // ---- merge my rows: the 8 partials in rank order, normalise, store as the output projection's activation tile ----
  const bool store = !*reinterpret_cast<volatile int*>(&suppress) && !*reinterpret_cast<volatile int*>(&abort_flag) &&
                     (n_me == 0 || *reinterpret_cast<volatile int*>(&mrg_ok));
  // per row: weight of every partial, already divided by the combined sum
  if (tid < HPC * n_me) {
    float ms[8], ls[8], mm = -INFINITY;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      const uint32_t blk = (s == rank) ? stg + (uint32_t)rank * L::SLOT : recv + (uint32_t)s * L::SLOT;
      asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(ms[s]), "=f"(ls[s]) : "r"(blk + (uint32_t)(HPC * n_me) * L::PITCH + (uint32_t)tid * 16) : "memory");
      mm = fmaxf(mm, ms[s]);
    }
    float w[8], ll = 0.f;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      w[s] = ms[s] == -INFINITY ? 0.f : exp2f(ms[s] - mm);
      ll = fmaf(w[s], ls[s], ll);
    }
    const float inv = 1.0f / ll;
#pragma unroll
    for (int s = 0; s < 8; ++s) wtab[tid][s] = w[s] * inv;
  }
  __syncthreads();
  if (store) {
    constexpr int CH = DH / 8;                // 16-byte chunks (8 columns) per row
    for (int idx = tid; idx < HPC * n_me * CH; idx += 288) {
      const int rr = idx / CH, ch = idx - rr * CH;       // rr = hl * n_me + il
      const int hl = rr >= n_me ? 1 : 0, il = rr - hl * n_me;
      float acc[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        const float w = wtab[rr][s];
        const uint32_t blk = (s == rank) ? stg + (uint32_t)rank * L::SLOT : recv + (uint32_t)s * L::SLOT;
        uint32_t u0, u1, u2, u3;
        asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(u0), "=r"(u1), "=r"(u2), "=r"(u3) : "r"(blk + (uint32_t)rr * L::PITCH + (uint32_t)ch * 16) : "memory");
        const uint32_t uu[4] = {u0, u1, u2, u3};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const __nv_bfloat162 p = *reinterpret_cast<const __nv_bfloat162*>(&uu[e]);
          acc[2 * e] = fmaf(w, __low2float(p), acc[2 * e]);
          acc[2 * e + 1] = fmaf(w, __high2float(p), acc[2 * e + 1]);
        }
      }
      const int orow = b * S + rank * 8 + il, col = (head0 + hl) * DH + ch * 8;
      *reinterpret_cast<uint4*>(a.out + out_index(orow, col, a.rows_pad, d.Nq)) =
          make_uint4(pack_bf16(acc[0], acc[1]), pack_bf16(acc[2], acc[3]), pack_bf16(acc[4], acc[5]), pack_bf16(acc[6], acc[7]));
    }
  }
  if (tracer) trace_stamp(trp, 5);
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  if (tracer) trace_stamp(trp, 6);
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem_base, COLS);
  }
  (void)base_ptr;
}

template <int DH, int HPC>
cudaError_t launch_one(const AttnArgs& a, int batch, cudaStream_t st) {
  static PerDeviceOnce once;
  if (once.needed()) {
    cudaError_t e = cudaFuncSetAttribute(k_attn_b1<DH, HPC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)B1Layout<DH, HPC>::SMEM);
    if (e != cudaSuccess) return e;
    once.done();
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(8, a.d.Hq / HPC, batch), cfg.blockDim = dim3(288), cfg.dynamicSmemBytes = B1Layout<DH, HPC>::SMEM, cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 8, at[0].val.clusterDim.y = 1, at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at, cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, k_attn_b1<DH, HPC>, a);
}

}  // namespace

// Two query heads per CTA must share a kv head; rotated bf16 operands only.
bool attention_b1_supported(const Dims& d) {
  return (d.dh == 256 || d.dh == 128) && d.S <= 64 && d.Hq % 2 == 0 && (d.Hq / d.Hkv) % 2 == 0;
}

// CTAs of one launch with `hpc` (1 or 2) query heads per CTA
int attention_b1_ctas(const Dims& d, int batch, int hpc) { return 8 * (d.Hq / hpc) * batch; }

cudaError_t launch_attention_b1(const Request* rq, int* status, const __nv_bfloat16* q_tiles, const __nv_bfloat16* kr,
                                const __nv_bfloat16* vr, int layer, __nv_bfloat16* out_tiled, int rows_pad, const Dims& d,
                                int batch, int hpc, unsigned wait_limit, cudaStream_t st, unsigned long long* trace, int trace_all) {
  AttnArgs a{};
  a.rq = rq, a.status = status, a.qr = q_tiles, a.kr = kr, a.vr = vr, a.layer = layer, a.out = out_tiled, a.rows_pad = rows_pad;
  a.num_splits = 8, a.d = d, a.wait_limit = wait_limit, a.trace = trace, a.trace_all = trace_all;
  if (hpc == 1) return d.dh == 256 ? launch_one<256, 1>(a, batch, st) : launch_one<128, 1>(a, batch, st);
  return d.dh == 256 ? launch_one<256, 2>(a, batch, st) : launch_one<128, 2>(a, batch, st);
}

}  // namespace phyai
