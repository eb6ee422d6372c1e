// The whole denoising loop of a small batch (batch * suffix_len <= 64 tokens) as ONE persistent
// kernel: every Euler step, every layer, the velocity head and the Euler update, with no host
// involvement and no kernel boundary in between.  (The paper captures the loop as a CUDA graph of
// many small kernels - graph-replay paragraph - and names a persistent "mega-kernel" as future work;
// this is that kernel, designed for sm_100a.)
//
// 148 CTAs (one per SM, cooperative launch so that all are resident) each own a fixed set of roles
// per layer - one GEMM tile per projection, a few attention (head pair, key range) roles, a row of a
// norm - and advance through the phases of a layer by waiting on global completion counters (bounded
// polls) instead of kernel boundaries.  Because a CTA's weight tiles are known in advance, four
// producer warps stream them through a shared-memory ring ahead of the dependency chain: HBM keeps
// flowing while the CTA waits for activations.
//
// Warp roles (512 threads): warps 0-7 workers (epilogues, attention, norms, head; 224 registers via
// setmaxnreg), warp 8 tcgen05 MMA issuer + TMEM owner, warps 9-10 activation producers, warps 11-15
// weight producers (32 registers).
//
// Shared memory: 9 x 16 KB weight ring (a CTA's next GEMM role is prefetched in full) + 64 KB
// "region A": two 32 KB slots through which the activations of the current GEMM role stream in chunks
// of four 64-wide k-chunks; the same 64 KB serve the attention role (Q tile + one K/V tile of 32 keys),
// the rotary / GeGLU exchange of the epilogues and the velocity head.  Its users take turns in program
// order.
#include "mega.h"

#include <algorithm>
#include <vector>

#include "attention.cuh"
#include "ptx.cuh"
#include "tc.cuh"

namespace phyai {
namespace {

constexpr int RING = 9;                 // weight ring slots
constexpr int UNIT = 16384;             // one weight block: 128 rows x 64 k, bf16
constexpr int ACT_TILE = 8192;          // one activation tile: 64 tokens x 64 k, bf16
constexpr int ACT_SLOT = 4 * ACT_TILE;   // activations stream through two slots of four k-chunks
constexpr int REGION_A = 2 * ACT_SLOT;
constexpr int KTA = 32;                 // keys per attention tile inside the persistent kernel
constexpr int NPROD_W = 5;              // weight producer warps (11..15)
constexpr int BAR_ATTN = 2;             // named barrier of the four attention warps
constexpr int NWORK = 256;              // worker threads
constexpr int BAR_WORK = 1;             // named barrier of the 8 worker warps
constexpr int MAX_D = 2048;
// tcgen05 instruction descriptor: D fp32, A/B bf16 K-major, N = 64, M = 128
constexpr uint32_t IDESC64 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(64 >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void work_sync() { group_sync<BAR_WORK, NWORK>(); }

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release(unsigned* p) {
  asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}
// Bounded wait until a completion counter reaches `target`.
__device__ __forceinline__ bool wait_count(const unsigned* ctr, unsigned target, const WaitCtx& c) {
  if (*c.abort_flag) return false;
  for (uint32_t it = 0; it < c.limit; ++it) {
    if (ld_acquire(ctr) >= target) return true;
    if (it > 64) __nanosleep(20);
  }
  *c.abort_flag = 1;
  atomicExch(c.status, ST_TIMEOUT);
  return false;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Trace stamp: which = 0 (worker: inputs ready / accumulator complete), 1 (worker: role done),
// 2 (MMA issuer: first activation chunk in shared memory), 3 (MMA issuer: last MMA issued).
__device__ __forceinline__ void stamp(const MegaParams& p, int phase, int step, int layer, int which, int wt) {
  if (p.trace && wt == 0 && step == p.trace_step && (layer == p.trace_layer || phase >= MP_EMBED))
    p.trace[((size_t)blockIdx.x * MP_COUNT + phase) * 4 + which] = global_ns();
}

struct Shared {
  uint64_t w_full[RING], w_empty[RING];
  uint64_t act_full[2], chunk_free[2];   // per activation slot
  uint64_t act_empty, acc_full, acc_empty;
  uint32_t tmem_slot;
  int abort_flag;
  int bcast;
  int tok_pos[64];   // rotary position of every suffix token: prefix_len of its request + index
  int tok_q[64];     // b * Hq * S + i   (row offset of the token in the rotated q buffer, before the head term)
  int tok_kv[64];    // b * Hkv * S + i
  int arow_out[64];  // residual-stream row of action row r: (r / H) * S + ns + r % H
  float red[16];
  float xs[64];
  alignas(16) float row[MAX_D];   // float4 accesses
};

// One entry of a CTA's program that uses region A: a GEMM role or the attention phase.
struct Item {
  bool gemm;
  int phase, step, layer;
  MegaGemmRole role;
};

// Enumerates, in execution order, the users of region A of this CTA.  Every agent (weight and
// activation producers, MMA issuer) walks the same sequence, so their slot and parity counters agree
// with the workers'.
struct ProgIter {
  const MegaParams& p;
  const MegaCtaPlan& pl;
  int step = 0, layer = 0, pos = -1;  // pos: -1 embed GEMM, 0 QKV, 1 ATTN, 2 O, 3 GATEUP, 4 DOWN
  bool started = false;
  __device__ ProgIter(const MegaParams& p_, const MegaCtaPlan& pl_) : p(p_), pl(pl_) {}
  __device__ bool next(Item& it) {
    for (;;) {
      if (!started) {
        started = true;
      } else if (++pos > 4) {
        pos = 0;
        if (++layer >= p.d.L) {
          layer = 0, pos = -1;
          if (++step >= p.n_steps) return false;
        }
      }
      if (step >= p.n_steps) return false;
      it.step = step, it.layer = layer;
      if (pos == -1) {
        if (pl.embed_gemm.kc_count > 0) {
          it.gemm = true, it.phase = MP_EMBED_GEMM, it.role = pl.embed_gemm;
          return true;
        }
      } else if (pos == 1) {
        if (pl.attn_end > pl.attn_begin) {
          it.gemm = false, it.phase = MP_ATTN;
          return true;
        }
      } else {
        const MegaGemmRole& c = pos == 0 ? pl.qkv : pos == 2 ? pl.o : pos == 3 ? pl.gateup : pl.down;
        if (c.kc_count > 0) {
          it.gemm = true, it.role = c;
          it.phase = pos == 0 ? MP_QKV : pos == 2 ? MP_O : pos == 3 ? MP_GATEUP : MP_DOWN;
          return true;
        }
      }
    }
  }
};

__device__ __forceinline__ const uint8_t* weight_base(const MegaParams& p, int phase, int layer) {
  switch (phase) {
    case MP_QKV: return reinterpret_cast<const uint8_t*>(p.w_qkv) + (size_t)layer * p.stride_qkv;
    case MP_O: return reinterpret_cast<const uint8_t*>(p.w_o) + (size_t)layer * p.stride_o;
    case MP_GATEUP: return reinterpret_cast<const uint8_t*>(p.w_gu) + (size_t)layer * p.stride_gu;
    case MP_DOWN: return reinterpret_cast<const uint8_t*>(p.w_d) + (size_t)layer * p.stride_d;
    default: return reinterpret_cast<const uint8_t*>(p.w_embed);
  }
}
__device__ __forceinline__ int phase_kc(const MegaParams& p, int phase) {
  return phase == MP_O ? p.d.Nq >> 6 : phase == MP_DOWN ? p.d.F >> 6 : p.d.D >> 6;
}
__device__ __forceinline__ const uint8_t* act_base(const MegaParams& p, int phase) {
  return reinterpret_cast<const uint8_t*>(phase == MP_O ? p.attn64
                                          : phase == MP_DOWN ? p.m64
                                          : phase == MP_EMBED_GEMM ? p.u64
                                                                   : p.xn64);
}
// Completion count the inputs of a GEMM role wait for.
__device__ __forceinline__ void gemm_dep(const MegaParams& p, int phase, int step, int layer, int& dep,
                                         unsigned& target) {
  const int inst = step * p.d.L + layer;
  switch (phase) {
    case MP_QKV: dep = MP_NORM1; break;
    case MP_O: dep = p.attn_splits > 1 ? MP_MERGE : MP_ATTN; break;
    case MP_GATEUP: dep = MP_NORM2; break;
    case MP_DOWN: dep = MP_GATEUP; break;
    default:
      dep = MP_EMBED;
      target = (unsigned)(step + 1) * (unsigned)p.n_cta[dep];
      return;
  }
  target = (unsigned)(inst + 1) * (unsigned)p.n_cta[dep];
}

__device__ __forceinline__ void site_params(const MegaParams& p, int step, int site, const float*& gain,
                                            const float*& shift, const float*& gate) {
  const int D = p.d.D;
  if (p.ada) {
    const float* base = p.mod + ((size_t)step * p.sites + site) * 3 * D;
    gain = base, shift = base + D, gate = base + 2 * D;
  } else {
    gain = p.gains + (size_t)site * D, shift = nullptr, gate = nullptr;
  }
}

// Residual reduction + (Ada)RMSNorm of one row by the 256 worker threads:
//   h[row] += sum of the `nslabs` split-K partial sums of the projection that precedes the norm,
//   out = h * rsqrt(mean h^2 + eps) * gain + shift -> tiled bf16 (rows_pad 64).
// The split-K partials are summed here, in a fixed order, instead of with atomics in the GEMM epilogue.
__device__ __forceinline__ void norm_row(const MegaParams& p, Shared& sh, int row, int nslabs, const float* gain,
                                         const float* shift, __nv_bfloat16* out, int wt) {
  const int D = p.d.D;
  float* x = p.h + (size_t)row * D;
  float ss = 0.f;
  for (int c = wt * 4; c < D; c += NWORK * 4) {
    float4 v = *reinterpret_cast<const float4*>(x + c);
    if (nslabs) {
      float4 part[8];
#pragma unroll
      for (int s = 0; s < 8; ++s)
        if (s < nslabs) part[s] = *reinterpret_cast<const float4*>(p.slab + ((size_t)s * 64 + row) * D + c);
#pragma unroll
      for (int s = 0; s < 8; ++s)
        if (s < nslabs) v.x += part[s].x, v.y += part[s].y, v.z += part[s].z, v.w += part[s].w;
      for (int s = 8; s < nslabs; ++s) {
        const float4 q = *reinterpret_cast<const float4*>(p.slab + ((size_t)s * 64 + row) * D + c);
        v.x += q.x, v.y += q.y, v.z += q.z, v.w += q.w;
      }
      *reinterpret_cast<float4*>(x + c) = v;
    }
    *reinterpret_cast<float4*>(sh.row + c) = v;
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = warp_sum(ss);
  if ((wt & 31) == 0) sh.red[wt >> 5] = ss;
  work_sync();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += sh.red[w];
  const float r = 1.0f / sqrtf(tot / (float)D + p.d.eps);
  if (out) {
    for (int c = wt * 4; c < D; c += NWORK * 4) {
      const float4 v = *reinterpret_cast<const float4*>(sh.row + c);   // written by this same thread
      const float4 g = *reinterpret_cast<const float4*>(gain + c);
      float4 o = make_float4(v.x * r * g.x, v.y * r * g.y, v.z * r * g.z, v.w * r * g.w);
      if (shift) {
        const float4 s4 = *reinterpret_cast<const float4*>(shift + c);
        o.x += s4.x, o.y += s4.y, o.z += s4.z, o.w += s4.w;
      }
      *reinterpret_cast<uint2*>(out + tiled_index(row, c, 64)) = make_uint2(pack_bf16(o.x, o.y), pack_bf16(o.z, o.w));
    }
  } else {   // keep the normalised row in shared memory (velocity head)
    for (int c = wt * 4; c < D; c += NWORK * 4) {
      float4 v = *reinterpret_cast<const float4*>(sh.row + c);
      const float4 g = *reinterpret_cast<const float4*>(gain + c);
      v = make_float4(v.x * r * g.x, v.y * r * g.y, v.z * r * g.z, v.w * r * g.w);
      if (shift) {
        const float4 s4 = *reinterpret_cast<const float4*>(shift + c);
        v.x += s4.x, v.y += s4.y, v.z += s4.z, v.w += s4.w;
      }
      *reinterpret_cast<float4*>(sh.row + c) = v;
    }
  }
  work_sync();  // sh.red / sh.row are reused by the next row
}

// Workers: signal that this CTA's part of `phase` is complete (all workers have finished their writes).
__device__ __forceinline__ void signal_phase(const MegaParams& p, int phase, int wt) {
  work_sync();
  if (wt == 0) {
    __threadfence();
    red_release(p.counters + phase);
  }
}
// Workers: wait until `phase` has completed `target` roles.  Returns the same value in every worker.
__device__ __forceinline__ bool await_phase(const MegaParams& p, Shared& sh, int phase, unsigned target,
                                            const WaitCtx& wc, int wt) {
  if (wt == 0) {
    sh.bcast = wait_count(p.counters + phase, target, wc) ? 1 : 0;
    __threadfence();
  }
  work_sync();
  const bool ok = sh.bcast != 0;
  work_sync();  // sh.bcast may be rewritten after this point
  return ok;
}

template <int DH>
__global__ void __launch_bounds__(512, 1) k_mega(const __grid_constant__ MegaParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ Shared sh;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const MegaCtaPlan& pl = p.plans[blockIdx.x];
  const Dims& d = p.d;
  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t regA = ring + RING * UNIT;
  float* regA_f = reinterpret_cast<float*>(smem_raw + (regA - smem_u32(smem_raw)));

  if (tid == 0) {
    sh.abort_flag = status_set(p.status) ? 1 : 0;
    for (int s = 0; s < RING; ++s) {
      mbar_init(smem_u32(&sh.w_full[s]), 1);
      mbar_init(smem_u32(&sh.w_empty[s]), 1);
    }
    for (int k = 0; k < 2; ++k) {
      mbar_init(smem_u32(&sh.act_full[k]), 1);
      mbar_init(smem_u32(&sh.chunk_free[k]), 1);
    }
    mbar_init(smem_u32(&sh.act_empty), 1);
    mbar_init(smem_u32(&sh.acc_full), 1);
    mbar_init(smem_u32(&sh.acc_empty), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    tmem_alloc(smem_u32(&sh.tmem_slot), 64);
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&sh.tmem_slot);
  const WaitCtx wc{p.status, &sh.abort_flag, p.wait_limit};
  if (sh.abort_flag) {   // the status word was already raised (failed validation): write nothing
    if (warp == 8) tmem_dealloc(tmem_base, 64);
    return;
  }

  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 32;");
    if (warp >= 11) {
      // ============ weight producers: unit u of the CTA's stream is loaded by warp 11 + u % 5 ================
      if (lane == 0) {
        ProgIter it(p, pl);
        Item im;
        unsigned u = 0;
        const unsigned me = (unsigned)(warp - 11);
        bool alive = true;
        while (alive && it.next(im)) {
          if (!im.gemm) continue;
          const uint8_t* src =
              weight_base(p, im.phase, im.layer) + ((size_t)im.role.tile * phase_kc(p, im.phase) + im.role.kc_begin) * UNIT;
          for (int j = 0; j < im.role.kc_count; ++j, ++u) {
            if (u % NPROD_W != me) continue;
            const unsigned s = u % RING, ph = (u / RING) & 1u;
            if (!mbar_wait(smem_u32(&sh.w_empty[s]), ph ^ 1u, wc)) {
              alive = false;
              break;
            }
            const uint32_t full = smem_u32(&sh.w_full[s]);
            mbar_expect_tx(full, UNIT);
            bulk_g2s(ring + s * UNIT, src + (size_t)j * UNIT, UNIT, full);
          }
        }
      }
    } else if (warp >= 9) {
      // ============ activation producers: warp 9 feeds slot 0, warp 10 slot 1; a role's k-chunks stream
      //              through the two slots in groups of four ==============================================
      if (lane == 0) {
        ProgIter it(p, pl);
        Item im;
        unsigned a_idx = 0;
        unsigned uses = 0;           // how many chunk groups this slot has received so far
        const int me = warp - 9;
        while (it.next(im)) {
          const unsigned a = a_idx++;
          if (!im.gemm) continue;
          if (a > 0) mbar_wait(smem_u32(&sh.act_empty), (a - 1) & 1u, wc);  // previous user released region A
          int dep;
          unsigned target;
          gemm_dep(p, im.phase, im.step, im.layer, dep, target);
          const bool ok = wait_count(p.counters + dep, target, wc);
          fence_async_proxy();
          const int groups = (im.role.kc_count + 3) / 4;
          for (int gidx = me; gidx < groups; gidx += 2, ++uses) {
            // within a role the slot is reused every other group: wait until the MMAs of its previous
            // occupant have finished reading it
            if (gidx >= 2) mbar_wait(smem_u32(&sh.chunk_free[me]), (uses - 1) & 1u, wc);
            const int j0 = gidx * 4, n = min(4, im.role.kc_count - j0);
            const uint32_t bytes = ok ? (uint32_t)n * ACT_TILE : 0u;
            const uint32_t full = smem_u32(&sh.act_full[me]);
            mbar_expect_tx(full, bytes);
            if (bytes)
              bulk_g2s(regA + (uint32_t)me * ACT_SLOT, act_base(p, im.phase) + (size_t)(im.role.kc_begin + j0) * ACT_TILE,
                       bytes, full);
          }
        }
      }
    } else if (warp == 8) {
      // ============ MMA issuer: the whole warp walks the program, one elected lane issues ==========================
      // A single warp issues roughly one instruction every few clocks, so the per-k-chunk body is kept
      // minimal: ring slot, parity and descriptors advance incrementally (no division), the weights of a
      // whole 4-chunk group are awaited up front, and the 16 MMAs of a group are issued back to back.
      {
        ProgIter it(p, pl);
        Item im;
        unsigned g = 0;
        unsigned uses0 = 0u, uses1 = 0u;   // chunk groups consumed from each activation slot
        unsigned ws = 0u, wph = 0u;        // weight ring slot and parity of the next unit
        const uint64_t da0 = make_desc(ring);
        const uint64_t db0 = make_desc(regA);
        while (it.next(im)) {
          if (!im.gemm) continue;
          bool ok = true;
          if (g > 0) ok = mbar_wait(smem_u32(&sh.acc_empty), (g - 1) & 1u, wc);  // epilogue drained TMEM
          const int groups = (im.role.kc_count + 3) >> 2;
          uint32_t accum = 0u;
          for (int gidx = 0; gidx < groups; ++gidx) {
            const int sl = gidx & 1;
            ok = mbar_wait(smem_u32(&sh.act_full[sl]), (sl ? uses1 : uses0) & 1u, wc) && ok;
            if (sl) ++uses1; else ++uses0;
            if (gidx == 0 && lane == 0) stamp(p, im.phase, im.step, im.layer, 2, 0);
            const int n = min(4, im.role.kc_count - gidx * 4);
            {   // all weight units of the group
              unsigned s2 = ws, ph2 = wph;
              for (int j = 0; j < n; ++j) {
                ok = mbar_wait(smem_u32(&sh.w_full[s2]), ph2, wc) && ok;
                if (++s2 == RING) s2 = 0, ph2 ^= 1u;
              }
            }
            tc_fence_after();
            const uint64_t db = db0 + (uint64_t)((sl * ACT_SLOT) >> 4);
            // a vote makes the condition provably warp-uniform, which keeps the descriptors below in
            // uniform registers (a branch on a value the compiler cannot prove uniform costs ~2x per MMA)
            if (__all_sync(0xffffffffu, ok)) {
              for (int j = 0; j < n; ++j) {
                const uint64_t da = da0 + (uint64_t)((ws * UNIT) >> 4);
                const uint64_t dbj = db + (uint64_t)((j * ACT_TILE) >> 4);
                if (elect_one()) {
                  umma_bf16(tmem_base, da, dbj, IDESC64, accum);
                  umma_bf16(tmem_base, da + 2, dbj + 2, IDESC64, 1u);
                  umma_bf16(tmem_base, da + 4, dbj + 4, IDESC64, 1u);
                  umma_bf16(tmem_base, da + 6, dbj + 6, IDESC64, 1u);
                  umma_commit(smem_u32(&sh.w_empty[ws]));
                }
                accum = 1u;
                if (++ws == RING) ws = 0, wph ^= 1u;
              }
            } else {
              for (int j = 0; j < n; ++j) {   // aborted: keep the ring protocol moving without issuing MMAs
                if (elect_one()) umma_commit(smem_u32(&sh.w_empty[ws]));
                if (++ws == RING) ws = 0, wph ^= 1u;
              }
            }
            if (elect_one()) umma_commit(smem_u32(&sh.chunk_free[sl]));   // the slot may be refilled
            __syncwarp();
          }
          if (lane == 0) stamp(p, im.phase, im.step, im.layer, 3, 0);
          if (elect_one()) umma_commit(smem_u32(&sh.acc_full));
          __syncwarp();
          ++g;
        }
      }
    }
  } else {
    // ================= workers ===============================================================================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
    const int wt = tid;                       // 0..255
    const int q = warp & 3, hf = warp >> 2;   // TMEM lane quarter, token-column half
    const Request rq = *p.rq;
    if (wt < 64) {   // per-token index tables: no integer division in the epilogue loops
      const int b = wt / d.S, i = wt % d.S;
      sh.tok_pos[wt] = wt < p.M ? rq.cu_lens[b + 1] - rq.cu_lens[b] + i : 0;
      sh.tok_q[wt] = b * d.Hq * d.S + i;
      sh.tok_kv[wt] = b * d.Hkv * d.S + i;
      sh.arow_out[wt] = (wt / d.H) * d.S + d.ns + wt % d.H;
    }
    work_sync();
    unsigned a_idx = 0, g_idx = 0;
    const int D = d.D, S = d.S, H = d.H;
    const int embed_last = p.ada ? MP_EMBED : MP_EMBED_GEMM;

    // ---- epilogue of one GEMM role ----
    auto epilogue = [&](const MegaGemmRole& r, int phase, int step, int layer) {
      if (wt == 0) sh.bcast = mbar_wait(smem_u32(&sh.acc_full), g_idx & 1u, wc) ? 1 : 0;
      work_sync();
      const bool ok = sh.bcast != 0;   // uniform over the workers: the barriers below must match
      stamp(p, phase, step, layer, 0, wt);
      tc_fence_after();
      const int ch = q * 32 + lane;           // row of the 128-row tile
      float v[32];
      tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(hf * 32), v);
      tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(hf * 32 + 16), v + 16);
      tc_fence_before();
      work_sync();
      if (wt == 0) mbar_arrive(smem_u32(&sh.acc_empty));   // the next role may overwrite the accumulator
      const int tok0 = hf * 32;
      if (ok) {
        if (phase == MP_QKV) {
          // rows 0..63 hold 64 channels of the first half of a head, rows 64..127 their rotary partners
          // (v tiles: plain order).  Exchange through shared memory, rotate, scale q, round to bf16.
          const int n = r.tile * 128 + ch;
          const float sc = p.s_qkv ? p.s_qkv[(size_t)layer * d.Nqkv + n] : 1.0f;
          const int Nk_end = d.Nq + d.Hkv * DH;
          const bool is_v = n >= Nk_end, is_q = n < d.Nq;
          const int c = is_v ? n : qkv_packed_to_channel(n, DH);     // channel in (q | k | v)
#pragma unroll
          for (int j = 0; j < 32; ++j) regA_f[(tok0 + j) * 128 + ch] = v[j] * sc;
          work_sync();
          constexpr int half = DH / 2;
          const int cin = is_q ? c % DH : (is_v ? (c - Nk_end) % DH : (c - d.Nq) % DH);   // channel within the head
          const int head = is_q ? c / DH : (is_v ? (c - Nk_end) / DH : (c - d.Nq) / DH);
          const int jrot = cin % half;
          const bool lower = cin < half;
          const float qs = is_q ? rsqrtf((float)DH) : 1.0f;
          const int partner = ch ^ 64;
          // two batches of 16 tokens: all table loads of a batch are issued before they are used
#pragma unroll
          for (int j0 = 0; j0 < 32; j0 += 16) {
            float2 cs[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int tok = tok0 + j0 + j;
              cs[j] = make_float2(1.f, 0.f);
              if (tok < p.M && !is_v && p.rope) cs[j] = p.rope[(size_t)sh.tok_pos[tok] * half + jrot];
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int tok = tok0 + j0 + j;
              if (tok < p.M) {
                const float other = regA_f[tok * 128 + partner];
                const float x = v[j0 + j] * sc;
                const float y = lower ? x * cs[j].x - other * cs[j].y : x * cs[j].x + other * cs[j].y;
                __nv_bfloat16* dst = is_q ? p.qr + (size_t)(sh.tok_q[tok] + head * S) * DH
                                          : (is_v ? p.vr : p.kr) + (size_t)(sh.tok_kv[tok] + head * S) * DH;
                dst[cin] = __float2bfloat16_rn(y * qs);
              }
            }
          }
        } else if (phase == MP_O || phase == MP_DOWN) {
          const int n = r.tile * 128 + ch;
          const float* sp = phase == MP_O ? p.s_o : p.s_d;
          float sc = sp ? sp[(size_t)layer * D + n] : 1.0f;
          if (p.ada) sc *= p.mod[(((size_t)step * p.sites + (2 * layer + (phase == MP_DOWN ? 1 : 0))) * 3 + 2) * D + n];
          float* dst = p.slab + (size_t)r.split * 64 * D + n;   // partial sums; the next norm adds them to h
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (tok0 + j < p.M) dst[(size_t)(tok0 + j) * D] = v[j] * sc;
        } else if (phase == MP_EMBED_GEMM) {
          const int n = r.tile * 128 + ch;
          const float bs = p.b2[n];
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int tok = tok0 + j;
            if (tok < p.batch * H) p.h[(size_t)sh.arow_out[tok] * D + n] = v[j] + bs;
          }
        } else {  // MP_GATEUP: rows 0..63 gate, rows 64..127 up of the same 64 channels
          const int c64 = ch & 63;
          const int f = r.tile * 64 + c64;
          if (q >= 2) {
            const float su = p.s_u ? p.s_u[(size_t)layer * d.F + f] : 1.0f;
#pragma unroll
            for (int j = 0; j < 32; ++j) regA_f[(tok0 + j) * 64 + c64] = v[j] * su;
          }
          work_sync();
          // the 64 x 64 bf16 result is exactly k-chunk `tile` of the down projection's input: build its
          // swizzled 8 KB image in shared memory, then copy it out with 16-byte stores
          __nv_bfloat16* img = reinterpret_cast<__nv_bfloat16*>(regA_f + 64 * 64);
          if (q < 2) {
            const float sg = p.s_g ? p.s_g[(size_t)layer * d.F + f] : 1.0f;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int tok = tok0 + j;
              const float m = gelu_fast(v[j] * sg, d.gelu_exact) * regA_f[tok * 64 + c64];
              img[tok * 64 + (((c64 >> 3) ^ (tok & 7)) << 3) + (c64 & 7)] = __float2bfloat16_rn(m);
            }
          }
          work_sync();
          uint4* gdst = reinterpret_cast<uint4*>(p.m64 + (size_t)r.tile * 64 * 64);
          const uint4* gsrc = reinterpret_cast<const uint4*>(img);
          for (int idx = wt; idx < 64 * 8; idx += NWORK)
            if ((idx >> 3) < p.M) gdst[idx] = gsrc[idx];
        }
      } else if (phase == MP_GATEUP) {
        work_sync();
        work_sync();
      } else if (phase == MP_QKV) {
        work_sync();
      }
      signal_phase(p, phase, wt);
      stamp(p, phase, step, layer, 1, wt);
      if (wt == 0) {
        fence_async_proxy();
        mbar_arrive(smem_u32(&sh.act_empty));   // region A is free for its next user
      }
      ++a_idx, ++g_idx;
    };

    for (int step = 0; step < p.n_steps; ++step) {
      // ---------------- suffix embedding ----------------
      if (pl.embed_end > pl.embed_begin) {
        if (step > 0) await_phase(p, sh, MP_FINAL, (unsigned)step * (unsigned)p.n_cta[MP_FINAL], wc, wt);
        stamp(p, MP_EMBED, step, 0, 0, wt);
        for (int r = pl.embed_begin; r < pl.embed_end; ++r) {
          const int b = r / H, i = r % H;
          if (wt < d.A) sh.xs[wt] = rq.x[(size_t)r * d.A + wt];
          work_sync();
          for (int n = wt * 4; n < D; n += NWORK * 4) {
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
            for (int a = 0; a < d.A; ++a) {
              const float4 w4 = *reinterpret_cast<const float4*>(p.Wc + (size_t)a * D + n);
              const float xa = sh.xs[a];
              acc.x = fmaf(xa, w4.x, acc.x), acc.y = fmaf(xa, w4.y, acc.y);
              acc.z = fmaf(xa, w4.z, acc.z), acc.w = fmaf(xa, w4.w, acc.w);
            }
            if (p.ada) {
              const float4 bb = *reinterpret_cast<const float4*>(p.bcfold + n);
              *reinterpret_cast<float4*>(p.h + (size_t)(b * S + d.ns + i) * D + n) =
                  make_float4(acc.x + bb.x, acc.y + bb.y, acc.z + bb.z, acc.w + bb.w);
            } else {
              const float4 tb = *reinterpret_cast<const float4*>(p.tb + (size_t)step * D + n);
              *reinterpret_cast<uint2*>(p.u64 + tiled_index(r, n, 64)) =
                  make_uint2(pack_bf16(swish_precise(acc.x + tb.x), swish_precise(acc.y + tb.y)),
                             pack_bf16(swish_precise(acc.z + tb.z), swish_precise(acc.w + tb.w)));
            }
            if (d.ns && i == 0)
              *reinterpret_cast<float4*>(p.h + (size_t)(b * S) * D + n) =
                  *reinterpret_cast<const float4*>(p.state_tok + (size_t)b * D + n);
          }
          work_sync();
        }
        signal_phase(p, MP_EMBED, wt);
        stamp(p, MP_EMBED, step, 0, 1, wt);
      }
      if (pl.embed_gemm.kc_count > 0) epilogue(pl.embed_gemm, MP_EMBED_GEMM, step, 0);

      for (int layer = 0; layer < d.L; ++layer) {
        const int inst = step * d.L + layer;
        const float *gain, *shift, *gate;
        // ---------------- norm 1 ----------------
        if (pl.norm_end > pl.norm_begin) {
          if (layer > 0)
            await_phase(p, sh, MP_DOWN, (unsigned)inst * (unsigned)p.n_cta[MP_DOWN], wc, wt);
          else
            await_phase(p, sh, embed_last, (unsigned)(step + 1) * (unsigned)p.n_cta[embed_last], wc, wt);
          stamp(p, MP_NORM1, step, layer, 0, wt);
          site_params(p, step, 2 * layer, gain, shift, gate);
          for (int row = pl.norm_begin; row < pl.norm_end; ++row)
            norm_row(p, sh, row, layer > 0 ? p.d_splits : 0, gain, shift, p.xn64, wt);
          signal_phase(p, MP_NORM1, wt);
          stamp(p, MP_NORM1, step, layer, 1, wt);
        }
        // ---------------- QKV ----------------
        if (pl.qkv.kc_count > 0) epilogue(pl.qkv, MP_QKV, step, layer);
        // ---------------- attention ----------------
        if (pl.attn_end > pl.attn_begin) {
          if (wt == 0 && a_idx > 0) mbar_wait(smem_u32(&sh.act_empty), (a_idx - 1) & 1u, wc);
          const bool go = await_phase(p, sh, MP_QKV, (unsigned)(inst + 1) * (unsigned)p.n_cta[MP_QKV], wc, wt);
          stamp(p, MP_ATTN, step, layer, 0, wt);
          AttnArgs a{};
          a.rq = p.rq, a.status = p.status, a.qkv = nullptr, a.rope = nullptr, a.layer = layer, a.out = p.attn64;
          a.qr = p.qr, a.kr = p.kr, a.vr = p.vr;
          a.rows_pad = 64, a.num_splits = p.attn_splits, a.part_o = p.attn_scratch;
          a.part_ml = p.attn_scratch + (size_t)p.batch * d.Hq * p.attn_splits * QROWS * DH;
          a.d = d, a.wait_limit = p.wait_limit;
          if (go && warp < 4) {   // one head per role, four warps; the other four workers wait at the barrier below
            for (int id = pl.attn_begin; id < pl.attn_end; ++id) {
              const int split = id % p.attn_splits, head = (id / p.attn_splits) % d.Hq, b = id / (p.attn_splits * d.Hq);
              attn_role<DH, 1, 1, BAR_ATTN, KTA>(a, split, head, b, regA, wt);
            }
          }
          signal_phase(p, MP_ATTN, wt);
          stamp(p, MP_ATTN, step, layer, 1, wt);
          if (wt == 0) {
            fence_async_proxy();
            mbar_arrive(smem_u32(&sh.act_empty));
          }
          ++a_idx;
        }
        // ---------------- merge of the split key ranges ----------------
        if (pl.merge_end > pl.merge_begin) {
          await_phase(p, sh, MP_ATTN, (unsigned)(inst + 1) * (unsigned)p.n_cta[MP_ATTN], wc, wt);
          stamp(p, MP_MERGE, step, layer, 0, wt);
          const float* part_o = p.attn_scratch;
          const float* part_ml = p.attn_scratch + (size_t)p.batch * d.Hq * p.attn_splits * QROWS * DH;
          for (int id = pl.merge_begin + warp; id < pl.merge_end; id += 8) {
            const int row = id % S, bh = id / S;   // bh = b * Hq + head
            const int b = bh / d.Hq, head = bh % d.Hq;
            const size_t slab0 = (size_t)bh * p.attn_splits * QROWS;
            // lane s holds (max, sum) of split s; weights 2^(m_s - m) / sum_s 2^(m_s - m) l_s by shuffles
            float ms = -INFINITY, ls = 0.f;
            if (lane < p.attn_splits) {
              const float2 ml = *reinterpret_cast<const float2*>(part_ml + (slab0 + (size_t)lane * QROWS + row) * 2);
              ms = ml.x, ls = ml.y;
            }
            const float mm = warp_max(ms);
            const float wgt = (ms == -INFINITY) ? 0.f : exp2f(ms - mm);
            const float inv = 1.0f / warp_sum(wgt * ls);
            constexpr int CPL = DH / 32;             // columns per lane
            float acc[CPL];
#pragma unroll
            for (int c = 0; c < CPL; ++c) acc[c] = 0.f;
            const float* src = part_o + (slab0 + row) * DH + lane * CPL;
#pragma unroll 4
            for (int s2 = 0; s2 < p.attn_splits; ++s2) {
              const float w = __shfl_sync(0xffffffffu, wgt, s2);
              float4 v4[CPL / 4];
#pragma unroll
              for (int c = 0; c < CPL / 4; ++c) v4[c] = *reinterpret_cast<const float4*>(src + (size_t)s2 * QROWS * DH + c * 4);
#pragma unroll
              for (int c = 0; c < CPL / 4; ++c) {
                acc[c * 4 + 0] = fmaf(w, v4[c].x, acc[c * 4 + 0]), acc[c * 4 + 1] = fmaf(w, v4[c].y, acc[c * 4 + 1]);
                acc[c * 4 + 2] = fmaf(w, v4[c].z, acc[c * 4 + 2]), acc[c * 4 + 3] = fmaf(w, v4[c].w, acc[c * 4 + 3]);
              }
            }
            __nv_bfloat16* dst = p.attn64 + tiled_index(b * S + row, head * DH + lane * CPL, 64);
#pragma unroll
            for (int c = 0; c < CPL; c += 2) *reinterpret_cast<uint32_t*>(dst + c) = pack_bf16(acc[c] * inv, acc[c + 1] * inv);
          }
          signal_phase(p, MP_MERGE, wt);
          stamp(p, MP_MERGE, step, layer, 1, wt);
        }
        // ---------------- O projection ----------------
        if (pl.o.kc_count > 0) epilogue(pl.o, MP_O, step, layer);
        // ---------------- norm 2 ----------------
        if (pl.norm_end > pl.norm_begin) {
          await_phase(p, sh, MP_O, (unsigned)(inst + 1) * (unsigned)p.n_cta[MP_O], wc, wt);
          stamp(p, MP_NORM2, step, layer, 0, wt);
          site_params(p, step, 2 * layer + 1, gain, shift, gate);
          for (int row = pl.norm_begin; row < pl.norm_end; ++row)
            norm_row(p, sh, row, p.o_splits, gain, shift, p.xn64, wt);
          signal_phase(p, MP_NORM2, wt);
          stamp(p, MP_NORM2, step, layer, 1, wt);
        }
        // ---------------- MLP ----------------
        if (pl.gateup.kc_count > 0) epilogue(pl.gateup, MP_GATEUP, step, layer);
        if (pl.down.kc_count > 0) epilogue(pl.down, MP_DOWN, step, layer);
      }

      // ---------------- final norm, velocity head, Euler update ----------------
      if (pl.final_end > pl.final_begin) {
        await_phase(p, sh, MP_DOWN, (unsigned)((step + 1) * d.L) * (unsigned)p.n_cta[MP_DOWN], wc, wt);
        stamp(p, MP_FINAL, step, 0, 0, wt);
        const float *gain, *shift, *gate;
        site_params(p, step, 2 * d.L, gain, shift, gate);
        for (int r = pl.final_begin; r < pl.final_end; ++r) {
          const int b = r / H, i = r % H;
          norm_row(p, sh, b * S + d.ns + i, p.d_splits, gain, shift, nullptr, wt);   // normalised row -> sh.row
          // v[a] = row . Wout[:, a]: thread (a, part) sums a slice of D, the parts combine in shared memory
          float* xo = rq.x + (size_t)r * d.A;
          const int parts = NWORK / 32;            // 8 slices of D per group of 32 outputs
          for (int a0 = 0; a0 < d.A; a0 += 32) {
            const int a = a0 + lane, part = warp;
            float acc = 0.f;
            if (a < d.A) {
              const int c0 = part * (D / parts), c1 = c0 + D / parts;
#pragma unroll 8
              for (int c = c0; c < c1; ++c) acc = fmaf(sh.row[c], p.Wout[(size_t)c * d.A + a], acc);
            }
            regA_f[part * 32 + lane] = acc;
            work_sync();
            if (warp == 0 && a < d.A) {
              float v = 0.f;
#pragma unroll
              for (int q2 = 0; q2 < parts; ++q2) v += regA_f[q2 * 32 + lane];
              xo[a] = xo[a] + p.dt * (v + p.bout[a]);
            }
            work_sync();
          }
        }
        signal_phase(p, MP_FINAL, wt);
        stamp(p, MP_FINAL, step, 0, 1, wt);
      }
    }
  }

  __syncthreads();
  if (sh.abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);  // let any copy still in flight land
  }
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 64);
  }
}

constexpr size_t MEGA_SMEM = 1024 + (size_t)RING * UNIT + REGION_A;

}  // namespace

// =============================================================================================
// host side
// =============================================================================================
bool mega_supported(const Dims& d, int batch) {
  if (batch * d.S > 64 || d.S > 64) return false;
  if (d.dh != 128 && d.dh != 256) return false;
  if (d.D % 128 || d.F % 64 || d.Nq % 128 || d.Nqkv % 128) return false;
  if (d.D > MAX_D || d.D / 64 > 16 || d.A > 64) return false;  // full-K roles hold <= 16 k-chunks in region A
  return true;
}

size_t mega_scratch_floats(const Dims& d, int batch, int splits) {
  return (size_t)batch * d.Hq * splits * QROWS * (d.dh + 2);
}

int mega_attention_splits(const Dims& d, int batch, int max_prefix, int ncta) {
  const int groups = batch * d.Hq;
  int want = ncta / groups;
  const int tiles = (max_prefix + KTA - 1) / KTA + (d.S + KTA - 1) / KTA;
  want = std::min(want, std::min(tiles, 16));
  return std::max(want, 1);
}

bool mega_plan(const Dims& d, int batch, int ada, int attn_splits, int ncta, MegaCtaPlan* plans, int* n_cta) {
  std::vector<int> load(ncta, 0);
  for (int c = 0; c < ncta; ++c) {
    plans[c] = MegaCtaPlan{};
  }
  for (int i = 0; i < MP_COUNT; ++i) n_cta[i] = 0;
  // GEMM roles: (tiles, k-chunks, k-split) per phase; each CTA holds at most one role of a phase.
  struct Ph { int phase, tiles, kc, splits; };
  auto splits_of = [](int kc) { return (kc + 7) / 8; };
  std::vector<Ph> phases = {
      {MP_GATEUP, d.F / 64, d.D / 64, 1},
      {MP_QKV, d.Nqkv / 128, d.D / 64, 1},
      {MP_DOWN, d.D / 128, d.F / 64, splits_of(d.F / 64)},
      {MP_O, d.D / 128, d.Nq / 64, splits_of(d.Nq / 64)},
  };
  if (!ada) phases.push_back({MP_EMBED_GEMM, d.D / 128, d.D / 64, 1});
  for (const Ph& ph : phases) {
    const int roles = ph.tiles * ph.splits;
    if (roles > ncta) return false;
    std::vector<char> used(ncta, 0);
    for (int r = 0; r < roles; ++r) {
      int best = -1;
      for (int c = 0; c < ncta; ++c)
        if (!used[c] && (best < 0 || load[c] < load[best])) best = c;
      used[best] = 1;
      const int tile = r / ph.splits, sp = r % ph.splits;
      MegaGemmRole role;
      role.tile = tile;
      role.kc_begin = ph.kc * sp / ph.splits;
      role.kc_count = ph.kc * (sp + 1) / ph.splits - role.kc_begin;
      role.split = sp;
      if (role.kc_count > 16 || role.kc_count < 1) return false;
      MegaCtaPlan& pl = plans[best];
      (ph.phase == MP_GATEUP ? pl.gateup : ph.phase == MP_QKV ? pl.qkv : ph.phase == MP_DOWN ? pl.down
       : ph.phase == MP_O ? pl.o : pl.embed_gemm) = role;
      load[best] += role.kc_count * (ph.phase == MP_EMBED_GEMM ? 0 : 1);
    }
    n_cta[ph.phase] = roles;
  }
  // row phases: one row per CTA, starting from the least loaded CTAs
  std::vector<int> order(ncta);
  for (int c = 0; c < ncta; ++c) order[c] = c;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return load[a] < load[b]; });
  const int M = batch * d.S, rowsA = batch * d.H;
  auto spread = [&](int n, auto set, int& count) {
    // contiguous ranges of ceil(n / ncta) rows over the CTAs in `order`
    const int per = (n + ncta - 1) / ncta;
    int r = 0;
    count = 0;
    for (int k = 0; k < ncta && r < n; ++k) {
      const int e = std::min(n, r + per);
      set(plans[order[k]], r, e);
      r = e;
      ++count;
    }
  };
  spread(M, [](MegaCtaPlan& pl, int b, int e) { pl.norm_begin = b, pl.norm_end = e; }, n_cta[MP_NORM1]);
  n_cta[MP_NORM2] = n_cta[MP_NORM1];
  spread(rowsA, [](MegaCtaPlan& pl, int b, int e) { pl.embed_begin = b, pl.embed_end = e; }, n_cta[MP_EMBED]);
  spread(rowsA, [](MegaCtaPlan& pl, int b, int e) { pl.final_begin = b, pl.final_end = e; }, n_cta[MP_FINAL]);
  // attention roles over all CTAs, least loaded first
  const int n_attn = batch * d.Hq * attn_splits;
  spread(n_attn, [](MegaCtaPlan& pl, int b, int e) { pl.attn_begin = b, pl.attn_end = e; }, n_cta[MP_ATTN]);
  if (attn_splits > 1) {
    const int n_merge = batch * d.Hq * d.S;
    // several rows per CTA (one per warp): ranges of up to ceil(n / ncta)
    spread(n_merge, [](MegaCtaPlan& pl, int b, int e) { pl.merge_begin = b, pl.merge_end = e; }, n_cta[MP_MERGE]);
  }
  return true;
}

cudaError_t mega_setup(int head_dim) {
  if (head_dim == 256)
    return cudaFuncSetAttribute(k_mega<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MEGA_SMEM);
  return cudaFuncSetAttribute(k_mega<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MEGA_SMEM);
}

cudaError_t launch_mega(const MegaParams& p, int ncta, cudaStream_t st) {
  void* args[] = {const_cast<MegaParams*>(&p)};
  const void* fn = p.d.dh == 256 ? (const void*)k_mega<256> : (const void*)k_mega<128>;
  return cudaLaunchCooperativeKernel(fn, dim3(ncta), dim3(512), args, MEGA_SMEM, st);
}

}  // namespace phyai
