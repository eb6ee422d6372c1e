// Host side of the C ABI: handle lifetime, weight repacking, per-step-count tables, the launch
// sequence of one denoising loop, CUDA-graph capture and replay.
#include <cstdarg>
#include <cstdio>
#include <algorithm>
#include <cstring>
#include <map>
#include <new>
#include <utility>
#include <vector>

#include "../../include/phyai.h"
#include "kernels.h"

using namespace phyai;

namespace {

thread_local char g_err[512] = "";

phyai_status_t fail(phyai_status_t code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

#define CU(call)                                                                                       \
  do {                                                                                                 \
    cudaError_t e_ = (call);                                                                           \
    if (e_ != cudaSuccess)                                                                             \
      return fail(e_ == cudaErrorMemoryAllocation ? PHYAI_ERR_OOM : PHYAI_ERR_CUDA, "%s failed: %s", #call, \
                  cudaGetErrorString(e_));                                                             \
  } while (0)

struct Tables {             // per n_steps
  float* tau = nullptr;     // [n][D]
  float* tb = nullptr;      // pi0:  [n][D]  time bias of the folded action MLP
  float* cvec = nullptr;    // pi05: [n][D]
  float* mod = nullptr;     // pi05: [n][sites][3D]  (1+scale | shift | gate)
  float* shw_qkv = nullptr; // pi05, cluster GEMM path: [n][L][Nqkv] shift . W_qkv in packed row order
  float* shw_gu = nullptr;  // pi05, cluster GEMM path: [n][L][2F]   shift . W_gate/up, interleaved row order
};

inline int kind_of(uint32_t dtype) { return dtype == PHYAI_F32 ? 0 : 1; }   // storage of everything but the big matrices

}  // namespace

struct phyai_expert {
  phyai_expert_config_t cfg{};
  Dims d{};
  bool tc = false;       // tensor-core engine
  bool ada = false;
  bool a8 = false;       // W8A8: e4m3 activations, FP8 tensor path (general kernels only)
  int sites = 0;
  int Mpad = 0;
  std::vector<void*> allocs;

  // small tensors (fp32)
  float *state_w = nullptr, *state_b = nullptr;
  float *Wc = nullptr;        // pi0: folded [A][D];  pi05: Wa [A][D]
  float *bcfold = nullptr;    // pi0: ba W1[0:D] + b1   pi05: ba
  float *W1tau = nullptr;     // pi0: W1[D:2D] fp32 [D][D]; pi05: W1 [D][D]
  float *b1 = nullptr, *W2f = nullptr, *b2 = nullptr;  // W2f: fp32 [D][D] (SIMT pi0 / pi05 table)
  __nv_bfloat16* W2p = nullptr;                        // TC pi0: packed
  float *Wout = nullptr, *bout = nullptr;
  float* gains = nullptr;      // plain: [sites][D] = 1 + gamma
  void* wmod = nullptr;        // ada: [sites][D][3D] in source storage
  float* bmod = nullptr;       // ada: [sites][3D]
  int wmod_kind = 0;

  // big matrices
  std::vector<float*> f_qkv, f_o, f_g, f_u, f_d;                 // SIMT fp32 row-major
  std::vector<__nv_bfloat16*> p_qkv, p_o, p_g, p_u, p_d;         // TC packed
  std::vector<float*> s_qkv, s_o, s_g, s_u, s_d;                 // TC per-channel scales (or null)
  std::vector<uint8_t*> b_qkv, b_o, b_gu, b_d;                   // e4m3 byte blocks for the cluster GEMM (W8 experts)

  float2* rope = nullptr;

  // workspace
  float *h = nullptr, *qkv = nullptr, *state_tok = nullptr;
  float *xn_f = nullptr, *attn_f = nullptr, *m_f = nullptr, *u_f = nullptr;
  __nv_bfloat16 *xn_t = nullptr, *attn_t = nullptr, *m_t = nullptr, *u_t = nullptr;

  float* attn_scratch = nullptr;  // split-KV partials of the tensor-core attention
  bool attn_mma = false;

  bool il_ok = false;          // gate / up also packed interleaved (single-token-tile calls)
  bool b1_ok = false;          // the cluster split-K GEMM path covers this expert's shapes
  int use_cluster_gemm = 1;
  int use_b1_attention = 1;
  int b1_attn_hpc = 0;         // query heads per CTA of the cluster attention kernel (0 = choose)
  int use_b1_step = 1;         // single-tile calls: velocity head + Euler update + next embedding as one cluster kernel
  int use_state_cache = 0;     // block-causal experts: state token computed once per call (single-tile calls); exact, but at
                               // one request the 18-layer state pass costs more than the 51st row it saves (measured)
  __nv_bfloat16 *kr_st = nullptr, *vr_st = nullptr;   // [L][max 64 tokens worth of requests][Hkv][S][dh] suffix K / V per layer
  int use_w8_inkernel = 1;     // e4m3 experts: the cluster GEMM decodes byte blocks itself (0: bf16 images made at create)    // tcgen05 attention with the key range split over a cluster (few requests)
  int b1_c[4] = {0, 0, 0, 0};  // cluster sizes of the QKV / O / gate-up / down projections (0 = choose)
  float *ss_a = nullptr, *ss_b = nullptr;   // [D/128][64] partial sums of squares of h (after O / after down)
  unsigned long long* trace_buf = nullptr;
  int trace_all_from = 0;                   // > 0: launches [from, from + 5) of a call trace every CTA
  unsigned long long* trace = nullptr;      // [TRACE_SLOTS][8] timer stamps of the traced launches of one call, or null
  int use_tc_attention = 1;
  int use_cluster_attention = 1;
  int use_fused_oproj = 1;     // cluster attention also does the output projection of its head (general GEMM path only)
  int n_sm = 0;
  __nv_bfloat16* p_gu_all = nullptr;        // gate/up interleaved in groups of 64 channels, all layers
  __nv_bfloat16* p_gu16 = nullptr;          // gate/up interleaved in groups of 16 channels (persistent tile GEMM)
  __nv_bfloat16* p_qkv16 = nullptr;         // q|k|v with the rows of every tile interleaved in groups of 16 (the same kernel)
  int use_persistent_gu = 1, use_persistent_qkv = 1, use_attn_splits = 1;
  float *s_qkv_all = nullptr, *s_o_all = nullptr, *s_g_all = nullptr, *s_u_all = nullptr, *s_d_all = nullptr;
  __nv_bfloat16 *xn64 = nullptr, *attn64 = nullptr, *m64 = nullptr, *u64 = nullptr;
  __nv_bfloat16 *qr64 = nullptr, *kr64 = nullptr, *vr64 = nullptr;
  uint8_t* xq = nullptr;     // W8A8: tiled e4m3 image of the current projection input [K/128][Mpad][128]
  float* xs = nullptr;       // W8A8: its per-token scales [Mpad]
  __nv_bfloat16* q_tiles = nullptr;   // cluster attention: q as [request][head pair][dh / 64][128 rows][64] swizzled tiles
  __nv_bfloat16 *qr_big = nullptr, *kr_big = nullptr, *vr_big = nullptr;   // rotated bf16 q / k / v of large batches

  Request* rq = nullptr;
  int* cu_internal = nullptr;
  int slab_splits = 8;         // most k-ranges a residual GEMM is split into when its partials go to slabs
  float* slab = nullptr;       // [MAX_SLABS][64][width] split-K partials of the residual GEMMs (one token tile)
  int* order = nullptr;        // requests by descending prefix length, rewritten by every batched call
  int* status = nullptr;

  std::map<int, Tables> tables;
  std::map<std::pair<int, int>, cudaGraphExec_t> graphs;
  std::map<std::pair<int, int>, uint64_t> launch_counts;
  cudaStream_t cap_stream = nullptr;

  // host-variant staging (allocated on first use)
  void* stg_kv = nullptr; size_t stg_kv_bytes = 0;
  float *stg_states = nullptr, *stg_noise = nullptr, *stg_out = nullptr;
  int* stg_cu = nullptr;

  int use_graph = 1;
  unsigned wait_limit = 1u << 22;
  uint64_t counting = 0;  // launches counted by the last enqueue

  template <typename T>
  phyai_status_t alloc(T** p, size_t count, bool zero = false) {
    void* q = nullptr;
    const size_t bytes = count * sizeof(T) > 0 ? count * sizeof(T) : 16;
    cudaError_t e = cudaMalloc(&q, bytes);
    if (e != cudaSuccess) return fail(PHYAI_ERR_OOM, "cudaMalloc(%zu bytes) failed: %s", bytes, cudaGetErrorString(e));
    allocs.push_back(q);
    if (zero) {
      e = cudaMemset(q, 0, bytes);
      if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "cudaMemset failed: %s", cudaGetErrorString(e));
    }
    *p = reinterpret_cast<T*>(q);
    return PHYAI_OK;
  }
};

#define ST(call)                         \
  do {                                   \
    phyai_status_t s_ = (call);          \
    if (s_ != PHYAI_OK) return s_;       \
  } while (0)

namespace {

size_t kv_elem_bytes(uint32_t dtype) { return dtype == PHYAI_F32 ? 4 : 2; }

phyai_status_t check_config(const phyai_expert_config_t* c) {
  if (!c) return fail(PHYAI_ERR_INVALID_ARG, "config is NULL");
  if (c->struct_size != sizeof(phyai_expert_config_t))
    return fail(PHYAI_ERR_INVALID_ARG, "config.struct_size %u != %zu", c->struct_size, sizeof(phyai_expert_config_t));
  if (!c->n_layers || !c->width || !c->mlp_dim || !c->n_q_heads || !c->n_kv_heads || !c->head_dim || !c->action_dim ||
      !c->horizon || !c->max_batch)
    return fail(PHYAI_ERR_INVALID_ARG, "a size in the config is zero");
  if (c->has_state_token > 1 || (c->has_state_token && !c->state_dim))
    return fail(PHYAI_ERR_INVALID_ARG, "has_state_token / state_dim inconsistent");
  if (c->n_q_heads % c->n_kv_heads) return fail(PHYAI_ERR_INVALID_ARG, "n_q_heads must be a multiple of n_kv_heads");
  if ((c->head_dim & 1) || (c->width & 1)) return fail(PHYAI_ERR_INVALID_ARG, "head_dim and width must be even");
  if (c->cond > PHYAI_COND_PI05_ADARMS || c->dtype > PHYAI_W4A16 || c->engine > PHYAI_ENGINE_SIMT)
    return fail(PHYAI_ERR_INVALID_ARG, "unknown cond / dtype / engine value");
  if (!(c->rms_eps >= 0.f) || !(c->rope_theta >= 0.f) || !(c->time_min_period > 0.f) || !(c->time_max_period > 0.f))
    return fail(PHYAI_ERR_INVALID_ARG, "rms_eps / rope_theta / time periods out of range");
  if (c->head_dim > 256) return fail(PHYAI_ERR_UNSUPPORTED, "head_dim > 256 is not covered");
  if ((uint64_t)c->max_batch * (c->horizon + c->has_state_token) > (1u << 22))
    return fail(PHYAI_ERR_UNSUPPORTED, "max_batch * suffix_len too large");
  return PHYAI_OK;
}

bool tc_shape_ok(const phyai_expert_config_t* c) {
  const uint32_t nq = c->n_q_heads * c->head_dim, nqkv = (c->n_q_heads + 2 * c->n_kv_heads) * c->head_dim;
  return c->width % 128 == 0 && c->mlp_dim % 128 == 0 && nq % 128 == 0 && nqkv % 128 == 0;
}

// ---------------------------------------------------------------------------------------------
// tables for one n_steps (time grid, sinusoid, pi0 time bias / pi0.5 modulation)
// ---------------------------------------------------------------------------------------------
phyai_status_t build_tables(phyai_expert* h, int n, cudaStream_t st, Tables** out) {
  auto it = h->tables.find(n);
  if (it != h->tables.end()) {
    *out = &it->second;
    return PHYAI_OK;
  }
  if (h->tables.size() >= 16) return fail(PHYAI_ERR_UNSUPPORTED, "more than 16 distinct n_steps on one handle");
  const int D = h->d.D;
  Tables t;
  ST(h->alloc(&t.tau, (size_t)n * D));
  launch_sinusoid(t.tau, n, D, (double)h->cfg.time_min_period, (double)h->cfg.time_max_period, st);
  if (!h->ada) {
    ST(h->alloc(&t.tb, (size_t)n * D));
    // tb_k = tau_k W1[D:2D] + (b1 + ba W1[0:D])
    launch_rows_gemm(t.tau, D, h->W1tau, 0, 0, D, D, h->bcfold, nullptr, 0, t.tb, D, n, st);
  } else {
    float* hid = nullptr;
    ST(h->alloc(&hid, (size_t)n * D));
    ST(h->alloc(&t.cvec, (size_t)n * D));
    ST(h->alloc(&t.mod, (size_t)n * h->sites * 3 * D));
    launch_rows_gemm(t.tau, D, h->W1tau, 0, 0, D, D, h->b1, nullptr, 1, hid, D, n, st);
    launch_rows_gemm(hid, D, h->W2f, 0, 0, D, D, h->b2, nullptr, 1, t.cvec, D, n, st);
    const size_t wsite = (size_t)D * 3 * D * (h->wmod_kind == 0 ? 4 : 2);
    for (int s = 0; s < h->sites; ++s)
      launch_rows_gemm(t.cvec, D, reinterpret_cast<const uint8_t*>(h->wmod) + s * wsite, h->wmod_kind, 0, 3 * D, D,
                       h->bmod + (size_t)s * 3 * D, nullptr, 0, t.mod + (size_t)s * 3 * D, h->sites * 3 * D, n, st);
    launch_mod_finish(t.mod, n * h->sites, D, st);
    if (h->b1_ok) {
      // the shift of a folded norm enters the projection after it as a per-channel constant shift . W
      const int L = h->d.L, Nqkv = h->d.Nqkv, F2 = 2 * h->d.F;
      ST(h->alloc(&t.shw_qkv, (size_t)n * L * Nqkv));
      ST(h->alloc(&t.shw_gu, (size_t)n * L * F2));
      for (int k = 0; k < n; ++k)
        for (int l = 0; l < L; ++l) {
          const float* sh1 = t.mod + ((size_t)k * h->sites + 2 * l) * 3 * D + D;
          const float* sh2 = t.mod + ((size_t)k * h->sites + 2 * l + 1) * 3 * D + D;
          launch_shift_rows(sh1, h->p_qkv[l], h->s_qkv[l], nullptr, 0, t.shw_qkv + ((size_t)k * L + l) * Nqkv, Nqkv, D, st);
          launch_shift_rows(sh2, h->p_gu_all + (size_t)l * D * F2, h->s_g[l], h->s_u[l], 1,
                            t.shw_gu + ((size_t)k * L + l) * F2, F2, D, st);
        }
    }
  }
  CU(cudaGetLastError());
  auto ins = h->tables.emplace(n, t);
  *out = &ins.first->second;
  return PHYAI_OK;
}

// ---------------------------------------------------------------------------------------------
// the loop: launches of one denoise call (x <- noise; n x [embed, L layers, head + Euler])
// ---------------------------------------------------------------------------------------------
// The tcgen05 attention kernel walks all keys of a request in one CTA per pair of query heads (no key split, no
// merge pass): from this many CTAs on it beats the split mma.sync kernel + merge.
constexpr int ATTN_TC_MIN_CTAS = 8;
constexpr int MAX_SLABS = 16;
constexpr int TRACE_SLOTS = 4096, TRACE_STAMPS = 16;

int pick_nt(int M) { return M <= 64 ? 64 : (M <= 1024 ? 128 : 256); }

// Token-tile width and split-K factor of a residual GEMM (N = width, large token counts): the pair that minimises
// waves x (k-chunks per CTA x clocks per k-chunk + epilogue).  The constants are a fit to launch durations (they
// put part of the exposed set-up and epilogue into the k-chunk term: the main loop alone runs at ~1180 clocks per
// 64 KB k-chunk); the choice they make for the pi-shaped expert at 64 requests, 192-token tiles with two k-ranges,
// is the measured optimum.
void pick_resid_tiling(int M, int Mpad, int N, int KC, int n_sm, int* nt_out, int* splits_out) {
  const int nts[2] = {256, 192};
  double best = 1e30;
  *nt_out = 256, *splits_out = 1;
  for (int nt : nts) {
    const int tok_tiles = (M + nt - 1) / nt;
    if (tok_tiles * nt > Mpad || N % 256) continue;
    for (int s = 1; s <= 4 && s <= KC; s *= 2) {
      const int ctas = tok_tiles * (N / 256) * s;
      const int waves = (ctas + n_sm - 1) / n_sm;
      const double per_kc = nt == 256 ? 1640.0 : 1436.0, epi = (s > 1 ? 9000.0 : 11000.0) * nt / 256.0 + 4000.0;
      const double cost = waves * ((double)((KC + s - 1) / s) * per_kc + epi);
      if (cost < best) best = cost, *nt_out = nt, *splits_out = s;
    }
  }
}

int pick_splits(int n_tiles, int tok_tiles, int KC) {
  int want = 148 / (n_tiles * tok_tiles);
  int s = 1;
  while (s * 2 <= want && s * 2 <= KC) s *= 2;
  return s;
}

phyai_status_t enqueue_loop(phyai_expert* h, int batch, int n, const Tables& t, cudaStream_t st) {
  const Dims& d0 = h->d;
  // State-token caching (block-causal suffix mask, plain norms): the state token sees the prefix and itself only, so
  // its hidden states and its rotated key / value of every layer depend neither on x nor on t.  They are computed
  // once per call by a pass over the state tokens alone and kept as key row 0 of every layer's suffix K / V; the
  // loop then runs on the action tokens only (query row i = key row 1 + i).  Single-tile calls on the cluster path.
  // A single 64-token tile: the projections run on the cluster split-K kernel with the norms folded in (five
  // kernels per layer: QKV, attention, O, gate/up, down).
  const bool b1_attn_tc = h->attn_mma && h->use_tc_attention && h->qr_big && attention_tc_supported(d0) &&
                          batch * (d0.Hq / 2) >= ATTN_TC_MIN_CTAS;
  const bool b1_attn_cluster = !b1_attn_tc && h->attn_mma && h->use_cluster_attention && batch * d0.Hq * 8 <= 2 * h->n_sm;
  const bool b1 = h->b1_ok && h->use_cluster_gemm && batch * d0.S <= 64 && (b1_attn_tc || b1_attn_cluster);
  const bool b1_attn_b1 = !b1_attn_tc && h->use_b1_attention && h->q_tiles && attention_b1_supported(d0) && batch * (d0.Hq / 2) * 8 <= h->n_sm;
  // one query head per CTA while the attention kernel then still leaves the QKV projection room beside it (the partial
  // results that cross the cluster, the softmax rows and the Q tile of a CTA halve), else two heads per CTA
  const int b1_hpc = (h->b1_attn_hpc == 1 || h->b1_attn_hpc == 2) ? h->b1_attn_hpc
                                                                 : (attention_b1_ctas(d0, batch, 1) <= h->n_sm / 2 ? 1 : 2);
  const bool cache_state = b1 && b1_attn_b1 && h->kr_st && h->use_state_cache;
  Dims d = d0;
  if (cache_state) d.ns = 0, d.S = d0.H, d.block_causal = 0, d.Sk = d0.S, d.Sk_stride = d0.S, d.koff = 1;
  const int M = batch * d.S, D = d.D;
  const int nt = pick_nt(M);
  const int tok_tiles = (M + nt - 1) / nt;
  const float dt = -1.0f / (float)n;
  uint64_t cnt = 0;
  auto site = [&](int k, int s, const float** gain, const float** shift, const float** gate) {
    if (h->ada) {
      const float* base = t.mod + ((size_t)k * h->sites + s) * 3 * D;
      *gain = base, *shift = base + D, *gate = base + 2 * D;
    } else {
      *gain = h->gains + (size_t)s * D, *shift = nullptr, *gate = nullptr;
    }
  };
  // Split-K partial sums of the residual GEMMs at one token tile go to slabs that the next reader of h (a norm or
  // the velocity head) adds in a fixed order: no atomics, so a request gives the same bits every time.
  int pending_slabs = 0;
  auto take_slabs = [&]() {
    SlabSum sl{h->slab, pending_slabs, (size_t)M * D};
    pending_slabs = 0;
    return sl;
  };
  const bool norm_q8 = h->a8 && rmsnorm_quantizes(D);   // W8A8: the norms write their e4m3 quantization themselves
  auto tc_gemm = [&](TcGemm g, bool prequantized = false) -> phyai_status_t {
    g.rows_pad = h->Mpad, g.M = g.M ? g.M : M, g.wait_limit = h->wait_limit, g.gelu_exact = d.gelu_exact;
    if (h->a8) {
      // W8A8: the projection input goes through the per-token e4m3 quantization, the product onto the FP8 tensor path
      if (!prequantized) {
        launch_quant_rows(h->status, g.X, h->xq, h->xs, h->Mpad, g.M, g.K, st);
        ++cnt;
      }
      g.X = reinterpret_cast<const __nv_bfloat16*>(h->xq), g.fp8 = 1, g.xscale = h->xs;
    }
    if (g.epi == TC_RESID && g.splits > 1 && nt == 64 && h->slab && D <= 2048) {
      if (g.splits > h->slab_splits) g.splits = h->slab_splits;
      g.slab = h->slab, pending_slabs = g.splits;
    }
    // trace_all_from = n: launch n of the call, if it is a tile GEMM, stamps one slot per CTA
    const long n_cta = (long)(g.N / 128) * ((g.M + 63) / 64) * (g.splits > 0 ? g.splits : 1);
    g.trace = (h->trace && h->trace_all_from > 0 && cnt == h->trace_all_from && n_cta <= TRACE_SLOTS) ? h->trace : nullptr;
    cudaError_t e = launch_tc_gemm(h->status, g, g.nt_override ? g.nt_override : nt, st);
    if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "tensor GEMM launch failed: %s", cudaGetErrorString(e));
    ++cnt;
    return PHYAI_OK;
  };
  auto simt_gemm = [&](SimtGemm g) {
    if (!g.rows_in) g.rows_in = g.rows_out = 1 << 30, g.row_off = 0;
    g.gelu_exact = d.gelu_exact;
    launch_simt_gemm(h->status, g, st);
    ++cnt;
  };

  const int kcb = h->a8 ? 128 : 64;   // contraction elements per 128-byte operand row (k-chunk of the tile GEMM)
  const int ss_n = D / 128;
  int trace_cursor = 0;
  const bool use_w8 = h->use_w8_inkernel && !h->b_qkv.empty();
  auto b1_gemm = [&](B1Gemm g, int which, int Mloc) -> phyai_status_t {
    g.M = Mloc, g.wait_limit = h->wait_limit, g.gelu_exact = d.gelu_exact, g.inv_D = 1.0f / (float)D, g.eps = d.eps;
    g.w_bits = h->cfg.dtype == PHYAI_W4A16 ? 4 : 8;
    g.trace = (h->trace && cnt < TRACE_SLOTS) ? h->trace + cnt * TRACE_STAMPS : nullptr;
    // The QKV projection leaves the SMs of the attention kernel free: that kernel then starts (and fetches its prefix
    // tiles) while the projection still runs.  Measured on the pi0-shaped expert: 7.6 ms per chunk with 140 CTAs,
    // 6.6 ms with 80 - 120.
    const int reserve = (which == 0 && b1_attn_b1) ? attention_b1_ctas(d, batch, b1_hpc) : 0;
    int C = b1_pick_cluster(g.N / 128, g.K / 64, h->n_sm - reserve);
    if (which == 0) {
      // Fewer, longer k-ranges for the QKV projection (about six k-chunks per CTA): all of its CTAs then find a free SM
      // while the previous layer's down projection still runs, and the reduce has fewer partials.  Measured on the
      // pi0-shaped expert: 6.31 ms per chunk with 5 k-ranges (100 CTAs), 6.23 ms with 3 (60 CTAs).
      const int c6 = (g.K / 64 + 5) / 6;
      if (c6 >= 1 && c6 < C && b1_gemm_supported(g.N, g.K, c6, h->n_sm, true)) C = c6;
    }
    if (h->b1_c[which] > 0 && b1_gemm_supported(g.N, g.K, h->b1_c[which], h->n_sm, which == 0)) C = h->b1_c[which];
    if (h->trace && h->trace_all_from > 0) {
      // every CTA of five consecutive launches stamps, one slot per CTA in launch order
      g.trace = nullptr;
      const int n_cta = C * (g.N / 128);
      if (cnt >= h->trace_all_from && cnt < h->trace_all_from + 5 && trace_cursor + n_cta <= TRACE_SLOTS) {
        g.trace = h->trace + (size_t)trace_cursor * TRACE_STAMPS, g.trace_all = 1;
        trace_cursor += n_cta;
      }
    }
    cudaError_t e = launch_b1_gemm(h->status, g, C, st);
    if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "cluster GEMM launch failed: %s", cudaGetErrorString(e));
    ++cnt;
    return PHYAI_OK;
  };

  // One layer on the cluster path: QKV, attention, O, gate/up, down (five kernels; the norms are folded in).
  // `kv_only`: stop after the QKV projection (the state pass needs nothing but the last layer's key / value).
  const size_t kv_layer = (size_t)batch * d0.Hkv * d0.S * d0.dh;   // per-layer stride of the cached suffix K / V
  auto b1_layer = [&](const Dims& dd, int Mloc, int k, int l, bool kv_only, __nv_bfloat16* kr, __nv_bfloat16* vr,
                      bool folded_first = false) -> phyai_status_t {
    const float *gain, *shift, *gate;
    site(k, 2 * l, &gain, &shift, &gate);
    // ---- QKV: layer 0 reads a normalised tile (or, `folded_first`, what the embedding kernels left); later layers
    // read bf16(h * gain) and the partial sums of squares left by the previous layer's down projection
    if (l == 0 && !folded_first) {
      launch_rmsnorm(h->status, h->h, gain, shift, nullptr, h->xn64, 64, Mloc, D, dd.eps, st);
      ++cnt;
    }
    B1Gemm q{};
    q.W = h->p_qkv[l], q.W8 = use_w8 ? h->b_qkv[l] : nullptr, q.X = h->xn64, q.N = dd.Nqkv, q.K = D, q.epi = B1_QKV, q.wscale = h->s_qkv[l];
    if (l > 0 || folded_first) {
      q.ss_part = h->ss_b, q.ss_n = ss_n;
      q.shift_row = h->ada ? t.shw_qkv + ((size_t)k * dd.L + l) * dd.Nqkv : nullptr;
    }
    q.rq = h->rq, q.rope = h->rope, q.qr = h->qr_big, q.kr = kr, q.vr = vr;
    q.q_tiles = b1_attn_b1 ? h->q_tiles : nullptr;
    q.S = dd.S, q.Hq = dd.Hq, q.Hkv = dd.Hkv, q.dh = dd.dh, q.Sk_stride = suffix_key_stride(dd), q.koff = dd.koff;
    ST(b1_gemm(q, 0, Mloc));
    if (kv_only) return PHYAI_OK;
    // ---- attention -> bf16 tile of the output projection
    cudaError_t e;
    if (b1_attn_b1) {
      unsigned long long* atr = (h->trace && !h->trace_all_from && cnt < TRACE_SLOTS) ? h->trace + cnt * TRACE_STAMPS : nullptr;
      int all = 0;
      const int n_cta = attention_b1_ctas(dd, batch, b1_hpc);
      if (h->trace && h->trace_all_from > 0 && cnt >= h->trace_all_from && cnt < h->trace_all_from + 5 &&
          trace_cursor + n_cta <= TRACE_SLOTS) {
        atr = h->trace + (size_t)trace_cursor * TRACE_STAMPS, all = 1;
        trace_cursor += n_cta;
      }
      e = launch_attention_b1(h->rq, h->status, h->q_tiles, kr, vr, l, h->attn64, 64, dd, batch, b1_hpc, h->wait_limit, st, atr, all);
    }
    else if (b1_attn_tc)
      e = launch_attention_tc(h->rq, h->status, h->qr_big, kr, vr, l, h->attn64, 64, dd, batch, h->order, h->wait_limit, st);
    else
      e = launch_attention_cluster(h->rq, h->status, h->qkv, h->rope, h->qr_big, kr, vr, l, h->attn64, 64, dd, batch,
                                   h->wait_limit, st, nullptr,
                                   (h->trace && !h->trace_all_from && cnt < TRACE_SLOTS) ? h->trace + cnt * TRACE_STAMPS : nullptr);
    if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "attention launch failed: %s", cudaGetErrorString(e));
    ++cnt;
    // ---- O projection + residual; leaves the operands of the second norm
    const float *gain2, *shift2, *gate2;
    site(k, 2 * l + 1, &gain2, &shift2, &gate2);
    B1Gemm o{};
    o.W = h->p_o[l], o.W8 = use_w8 ? h->b_o[l] : nullptr, o.X = h->attn64, o.N = D, o.K = dd.Nq, o.epi = B1_RESID, o.wscale = h->s_o[l];
    o.h = h->h, o.ldh = D, o.gate = gate, o.gain_next = gain2, o.xn_out = h->xn64, o.ss_out = h->ss_a;
    ST(b1_gemm(o, 1, Mloc));
    // ---- gate / up + GeGLU
    B1Gemm gu{};
    gu.W = h->p_gu_all + (size_t)l * D * 2 * dd.F, gu.W8 = use_w8 ? h->b_gu[l] : nullptr, gu.X = h->xn64, gu.N = 2 * dd.F, gu.K = D, gu.epi = B1_GEGLU;
    gu.wscale = h->s_g[l], gu.wscale2 = h->s_u[l], gu.ss_part = h->ss_a, gu.ss_n = ss_n;
    gu.shift_row = h->ada ? t.shw_gu + ((size_t)k * dd.L + l) * 2 * dd.F : nullptr;
    gu.out_tiled = h->m64;
    ST(b1_gemm(gu, 2, Mloc));
    // ---- down projection + residual; leaves the operands of the next layer's first norm
    B1Gemm dn{};
    dn.W = h->p_d[l], dn.W8 = use_w8 ? h->b_d[l] : nullptr, dn.X = h->m64, dn.N = D, dn.K = dd.F, dn.epi = B1_RESID, dn.wscale = h->s_d[l];
    dn.h = h->h, dn.ldh = D, dn.gate = gate2;
    if (l + 1 < dd.L) {
      const float *gain3, *shift3, *gate3;
      site(k, 2 * l + 2, &gain3, &shift3, &gate3);
      dn.gain_next = gain3, dn.xn_out = h->xn64, dn.ss_out = h->ss_b;
    }
    ST(b1_gemm(dn, 3, Mloc));
    return PHYAI_OK;
  };

  launch_begin(h->rq, h->status, h->state_w, h->state_b, h->state_tok, d0, batch, st);
  ++cnt;
  if (cache_state) {
    // the state tokens alone through every layer: row b of h = request b's state token
    Dims dp = d0;
    dp.S = 1, dp.Sk = 1, dp.Sk_stride = d0.S, dp.koff = 0;
    CU(cudaMemcpyAsync(h->h, h->state_tok, (size_t)batch * D * sizeof(float), cudaMemcpyDeviceToDevice, st));
    for (int l = 0; l < d0.L; ++l)
      ST(b1_layer(dp, batch, 0, l, l + 1 == d0.L, h->kr_st + (size_t)l * kv_layer, h->vr_st + (size_t)l * kv_layer));
  }
  // Single-tile calls: one cluster kernel per step boundary (velocity head and Euler update of step k - 1, embedding
  // of step k), then for pi0 the MLP's second layer on the cluster GEMM, whose epilogue leaves layer 0's norm operands.
  const bool b1_step = b1 && h->use_b1_step && h->tc && step_b1_supported(d, batch) && (h->ada || h->W2p);
  auto step_kernel = [&](int k, bool first, bool last) -> phyai_status_t {
    StepB1 p{};
    p.rq = h->rq, p.batch = batch, p.S = d.S, p.H = d.H, p.ns = d.ns, p.A = d.A, p.D = D, p.M = M, p.eps = d.eps;
    p.wait_limit = h->wait_limit, p.first = first, p.last = last, p.h_in = h->h, p.Wout = h->Wout, p.bout = h->bout, p.dt = dt;
    if (!first) {
      const float* gate_unused;
      site(k - 1, 2 * d.L, &p.gain_f, &p.shift_f, &gate_unused);
    }
    p.ada = h->ada ? 1 : 0, p.Wc = h->Wc, p.state_tok = h->state_tok;
    if (!last) {
      if (h->ada) {
        const float *shift0, *gate0;
        site(k, 0, &p.gain_next, &shift0, &gate0);
        p.bias = h->bcfold, p.h_out = h->h, p.xn_out = h->xn64, p.ss_out = h->ss_b;
      } else {
        p.bias = t.tb + (size_t)k * D, p.u = h->m64;
      }
    }
    p.trace = (h->trace && !h->trace_all_from && cnt < TRACE_SLOTS) ? h->trace + cnt * TRACE_STAMPS : nullptr;
    cudaError_t e = launch_step_b1(h->status, p, st);
    if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "step kernel launch failed: %s", cudaGetErrorString(e));
    ++cnt;
    return PHYAI_OK;
  };
  for (int k = 0; k < n; ++k) {
    // ---- suffix embedding ----
    if (b1_step) {
      ST(step_kernel(k, k == 0, false));
      if (!h->ada) {
        B1Gemm e{};
        e.W = h->W2p, e.X = h->m64, e.N = D, e.K = D, e.epi = B1_RESID, e.h = h->h, e.ldh = D;
        e.bias = h->b2, e.state_tok = h->state_tok, e.ns = d.ns, e.S = d.S;
        const float *shift0, *gate0;
        site(k, 0, &e.gain_next, &shift0, &gate0);
        e.xn_out = h->xn64, e.ss_out = h->ss_b;
        ST(b1_gemm(e, 1, M));
      }
    } else if (!h->ada) {
      launch_embed_pi0(h->rq, h->status, h->Wc, t.tb + (size_t)k * D, h->state_tok, h->h, h->u_f, h->u_t, h->Mpad, d,
                       batch, st);
      ++cnt;
      const int rows = batch * d.H;
      if (h->tc) {
        TcGemm g{};
        g.W = h->W2p, g.X = h->u_t, g.M = rows, g.N = D, g.K = D, g.epi = TC_BIAS_ROWMAP, g.bias = h->b2;
        g.out_f32 = h->h, g.ldo = D, g.rows_in = d.H, g.rows_out = d.S, g.row_off = d.ns, g.splits = 1;
        // token tiling of the action rows alone
        g.rows_pad = h->Mpad, g.wait_limit = h->wait_limit;
        cudaError_t e = launch_tc_gemm(h->status, g, pick_nt(rows), st);
        if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "tensor GEMM launch failed: %s", cudaGetErrorString(e));
        ++cnt;
      } else {
        SimtGemm g{};
        g.A = h->u_f, g.lda = D, g.B = h->W2f, g.M = rows, g.N = D, g.K = D, g.epi = EPI_STORE, g.bias = h->b2;
        g.out = h->h, g.ldo = D, g.rows_in = d.H, g.rows_out = d.S, g.row_off = d.ns;
        simt_gemm(g);
      }
    } else {
      launch_embed_pi05(h->rq, h->status, h->Wc, h->bcfold, h->state_tok, h->h, d, batch, st);
      ++cnt;
    }
    // ---- transformer layers ----
    for (int l = 0; l < d.L; ++l) {
      const float *gain, *shift, *gate;
      site(k, 2 * l, &gain, &shift, &gate);
      if (b1) {
        ST(b1_layer(d, M, k, l, false, cache_state ? h->kr_st + (size_t)l * kv_layer : h->kr_big,
                    cache_state ? h->vr_st + (size_t)l * kv_layer : h->vr_big, b1_step));
        continue;
      }
      launch_rmsnorm(h->status, h->h, gain, shift, h->xn_f, h->xn_t, h->Mpad, M, D, d.eps, st, take_slabs(),
                     norm_q8 ? h->xq : nullptr, norm_q8 ? h->xs : nullptr);
      ++cnt;
      const bool attn_tc = h->attn_mma && h->use_tc_attention && h->qr_big && attention_tc_supported(d) &&
                           batch * (d.Hq / 2) >= ATTN_TC_MIN_CTAS;
      const bool attn_cluster = !attn_tc && h->attn_mma && h->use_cluster_attention && batch * d.Hq * 8 <= 2 * h->n_sm;
      const bool attn_rot = h->qr_big && (attn_tc || attn_cluster);   // q / k / v leave the QKV epilogue rotated, bf16
      // one token tile: the cluster attention kernel multiplies each head's output by its slice of Wo itself and
      // writes one slab per head, which the next norm sums like the k-range partials of a split-K GEMM
      const bool fuse_o = attn_cluster && attn_rot && h->tc && !h->a8 && h->use_fused_oproj && h->slab && M <= 64 &&
                          d.Hq <= MAX_SLABS && attention_oproj_supported(d);
      if (h->tc) {
        TcGemm g{};
        g.W = h->p_qkv[l], g.X = h->xn_t, g.N = d.Nqkv, g.K = D, g.epi = TC_STORE, g.scale = h->s_qkv[l];
        g.perm_dh = d.dh, g.perm_end = d.Nq + d.Hkv * d.dh;
        g.out_f32 = h->qkv, g.ldo = d.Nqkv, g.splits = 1;
        if (attn_rot) {
          // these attention kernels take their operands rotated, scaled and rounded from this epilogue
          g.epi = TC_QKV_ROT, g.rq = h->rq, g.rope = h->rope, g.qr = h->qr_big, g.kr = h->kr_big, g.vr = h->vr_big;
          g.S = d.S, g.Hq = d.Hq, g.Hkv = d.Hkv, g.dh = d.dh;
        }
        if (attn_rot && nt == 256 && h->p_qkv16 && h->use_persistent_qkv && persist_gemm_supported(M, d.Nqkv, D, h->Mpad, h->a8)) {
          if (h->a8 && !norm_q8) {
            launch_quant_rows(h->status, h->xn_t, h->xq, h->xs, h->Mpad, M, D, st);
            ++cnt;
          }
          PersistGemm p{};
          p.W = h->p_qkv16 + (size_t)l * D * d.Nqkv / (h->a8 ? 2 : 1);
          p.X = h->a8 ? reinterpret_cast<const __nv_bfloat16*>(h->xq) : h->xn_t;
          p.scale_g = h->s_qkv[l], p.xscale = h->a8 ? h->xs : nullptr;
          p.M = M, p.N = d.Nqkv, p.K = D, p.rows_pad = h->Mpad, p.fp8 = h->a8 ? 1 : 0, p.qkv = 1;
          p.wait_limit = h->wait_limit;
          p.rq = h->rq, p.rope = h->rope, p.qr = h->qr_big, p.kr = h->kr_big, p.vr = h->vr_big;
          p.S = d.S, p.Hq = d.Hq, p.Hkv = d.Hkv, p.dh = d.dh;
          p.trace = (h->trace && h->trace_all_from > 0 && cnt == h->trace_all_from) ? h->trace : nullptr;
          cudaError_t e = launch_persist_gemm(h->status, p, h->n_sm, st);
          if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "q|k|v GEMM launch failed: %s", cudaGetErrorString(e));
          ++cnt;
        } else {
          ST(tc_gemm(g, norm_q8));
        }
      } else {
        SimtGemm g{};
        g.A = h->xn_f, g.lda = D, g.B = h->f_qkv[l], g.M = M, g.N = d.Nqkv, g.K = D, g.epi = EPI_STORE;
        g.out = h->qkv, g.ldo = d.Nqkv;
        simt_gemm(g);
      }
      if (attn_tc) {
        const int tsp = (h->use_attn_splits && h->attn_scratch) ? attention_tc_splits(d, batch, h->n_sm, (int)h->cfg.max_prefix_len) : 1;
        cudaError_t e = launch_attention_tc(h->rq, h->status, h->qr_big, h->kr_big, h->vr_big, l, h->attn_t, h->Mpad, d,
                                            batch, h->order, h->wait_limit, st,
                                            (h->trace && h->trace_all_from > 0 && cnt == h->trace_all_from && batch * (d.Hq / 2) * tsp <= TRACE_SLOTS) ? h->trace : nullptr,
                                            tsp, h->attn_scratch);
        if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "attention launch failed: %s", cudaGetErrorString(e));
        cnt += tsp > 1 ? 2 : 1;
      } else if (attn_cluster) {
        // few requests: 8 key ranges per head in a cluster of 8 CTAs, merged through distributed shared memory
        const AttnOproj op{h->p_o[l], h->s_o[l], gate, h->slab, (size_t)M * D};
        cudaError_t e = launch_attention_cluster(h->rq, h->status, h->qkv, h->rope, attn_rot ? h->qr_big : nullptr, h->kr_big,
                                                 h->vr_big, l, h->attn_t, h->Mpad, d, batch, h->wait_limit, st,
                                                 fuse_o ? &op : nullptr);
        if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "attention launch failed: %s", cudaGetErrorString(e));
        ++cnt;
        if (fuse_o) pending_slabs = d.Hq;
      } else if (h->attn_mma) {
        const int splits = attention_pick_splits(d, batch, (int)h->cfg.max_prefix_len);
        cudaError_t e = launch_attention_mma(h->rq, h->status, h->qkv, h->rope, l, h->attn_t, h->Mpad, splits,
                                             h->attn_scratch, d, batch, h->wait_limit, st);
        if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "attention launch failed: %s", cudaGetErrorString(e));
        cnt += splits > 1 ? 2 : 1;
      } else {
        launch_attention_simt(h->rq, h->status, h->qkv, h->rope, l, h->cfg.dtype != PHYAI_F32, h->attn_f, h->attn_t,
                              h->Mpad, d, batch, st);
        ++cnt;
      }
      if (fuse_o) {
        // (projected inside the attention kernel)
      } else if (h->tc) {
        TcGemm g{};
        g.W = h->p_o[l], g.X = h->attn_t, g.N = D, g.K = d.Nq, g.epi = TC_RESID, g.scale = h->s_o[l], g.gate = gate;
        g.out_f32 = h->h, g.ldo = D, g.splits = pick_splits(D / 128 / ((nt == 256 && D % 256 == 0) ? 2 : 1), tok_tiles, d.Nq / kcb);
        if (nt == 256 && D % 256 == 0) pick_resid_tiling(M, h->Mpad, D, d.Nq / kcb, h->n_sm, &g.nt_override, &g.splits);
        ST(tc_gemm(g));
      } else {
        SimtGemm g{};
        g.A = h->attn_f, g.lda = d.Nq, g.B = h->f_o[l], g.M = M, g.N = D, g.K = d.Nq, g.epi = EPI_RESID, g.gate = gate;
        g.out = h->h, g.ldo = D;
        simt_gemm(g);
      }
      site(k, 2 * l + 1, &gain, &shift, &gate);
      launch_rmsnorm(h->status, h->h, gain, shift, h->xn_f, h->xn_t, h->Mpad, M, D, d.eps, st, take_slabs(),
                     norm_q8 ? h->xq : nullptr, norm_q8 ? h->xs : nullptr);
      ++cnt;
      if (h->tc) {
        TcGemm g{};
        g.W = h->p_g[l], g.W2 = h->p_u[l], g.X = h->xn_t, g.N = d.F, g.K = D, g.epi = TC_GEGLU;
        g.scale = h->s_g[l], g.scale2 = h->s_u[l], g.out_tiled = h->m_t, g.splits = 1;
        if (nt == 64 && h->p_gu_all) {
          // a single token tile: interleaved gate / up tiles put the weight stream on twice as many SMs
          g.W = h->p_gu_all + (size_t)l * D * 2 * d.F, g.W2 = nullptr, g.N = 2 * d.F, g.epi = TC_GEGLU_IL;
        }
        if (nt == 256 && h->p_gu16 && h->use_persistent_gu && persist_gemm_supported(M, 2 * d.F, D, h->Mpad, h->a8)) {
          if (h->a8 && !norm_q8) {
            launch_quant_rows(h->status, h->xn_t, h->xq, h->xs, h->Mpad, M, D, st);
            ++cnt;
          }
          PersistGemm p{};
          p.W = h->p_gu16 + (size_t)l * D * 2 * d.F / (h->a8 ? 2 : 1);
          p.X = h->a8 ? reinterpret_cast<const __nv_bfloat16*>(h->xq) : h->xn_t;
          p.out_tiled = h->m_t, p.scale_g = h->s_g[l], p.scale_u = h->s_u[l], p.xscale = h->a8 ? h->xs : nullptr;
          p.M = M, p.N = 2 * d.F, p.K = D, p.rows_pad = h->Mpad, p.gelu_exact = d.gelu_exact, p.fp8 = h->a8 ? 1 : 0;
          p.wait_limit = h->wait_limit;
          p.trace = (h->trace && h->trace_all_from > 0 && cnt == h->trace_all_from) ? h->trace : nullptr;
          cudaError_t e = launch_persist_gemm(h->status, p, h->n_sm, st);
          if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "gate/up GEMM launch failed: %s", cudaGetErrorString(e));
          ++cnt;
        } else {
          ST(tc_gemm(g, norm_q8));
        }
        TcGemm g2{};
        g2.W = h->p_d[l], g2.X = h->m_t, g2.N = D, g2.K = d.F, g2.epi = TC_RESID, g2.scale = h->s_d[l], g2.gate = gate;
        g2.out_f32 = h->h, g2.ldo = D, g2.splits = pick_splits(D / 128 / ((nt == 256 && D % 256 == 0) ? 2 : 1), tok_tiles, d.F / kcb);
        if (nt == 256 && D % 256 == 0) pick_resid_tiling(M, h->Mpad, D, d.F / kcb, h->n_sm, &g2.nt_override, &g2.splits);
        ST(tc_gemm(g2));
      } else {
        SimtGemm g{};
        g.A = h->xn_f, g.lda = D, g.B = h->f_g[l], g.B2 = h->f_u[l], g.M = M, g.N = d.F, g.K = D, g.epi = EPI_GEGLU;
        g.out = h->m_f, g.ldo = d.F;
        simt_gemm(g);
        SimtGemm g2{};
        g2.A = h->m_f, g2.lda = d.F, g2.B = h->f_d[l], g2.M = M, g2.N = D, g2.K = d.F, g2.epi = EPI_RESID, g2.gate = gate;
        g2.out = h->h, g2.ldo = D;
        simt_gemm(g2);
      }
    }
    // ---- final norm, velocity head, Euler update ----
    if (b1_step) {
      if (k + 1 == n) ST(step_kernel(n, false, true));
      continue;
    }
    const float *gain, *shift, *gate;
    site(k, 2 * d.L, &gain, &shift, &gate);
    if (pending_slabs) {
      launch_add_slabs(h->status, h->h, M, D, st, take_slabs());
      ++cnt;
    }
    launch_final(h->rq, h->status, h->h, gain, shift, h->Wout, h->bout, dt, d, batch, st);
    ++cnt;
  }
  h->counting = cnt;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
  return PHYAI_OK;
}

phyai_status_t run(phyai_expert* h, const Request& r, int n, cudaStream_t st) {
  Tables* t = nullptr;
  ST(build_tables(h, n, st, &t));
  launch_set_request(h->rq, r, h->cu_internal, st, h->order);
  if (r.cu_lens != nullptr) launch_validate(h->rq, h->status, (int)h->cfg.max_prefix_len, h->order, st);
  const auto key = std::make_pair(r.batch, n);
  if (!h->use_graph) {
    ST(enqueue_loop(h, r.batch, n, *t, st));
    h->launch_counts[key] = h->counting;
    return PHYAI_OK;
  }
  auto it = h->graphs.find(key);
  if (it == h->graphs.end()) {
    if (h->graphs.size() >= 64) return fail(PHYAI_ERR_UNSUPPORTED, "more than 64 captured (batch, n_steps) graphs");
    // tables were enqueued on `st`; the capture stream must not run ahead of them on first replay,
    // which holds because the graph is launched on `st` below.
    cudaGraph_t graph = nullptr;
    CU(cudaStreamBeginCapture(h->cap_stream, cudaStreamCaptureModeThreadLocal));
    phyai_status_t s = enqueue_loop(h, r.batch, n, *t, h->cap_stream);
    cudaError_t e = cudaStreamEndCapture(h->cap_stream, &graph);
    if (s != PHYAI_OK) {
      if (graph) cudaGraphDestroy(graph);
      return s;
    }
    if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "graph capture failed: %s", cudaGetErrorString(e));
    cudaGraphExec_t exec = nullptr;
    e = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) return fail(PHYAI_ERR_CUDA, "graph instantiate failed: %s", cudaGetErrorString(e));
    it = h->graphs.emplace(key, exec).first;
    h->launch_counts[key] = h->counting;
  }
  CU(cudaGraphLaunch(it->second, st));
  return PHYAI_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

phyai_status_t check_call(phyai_expert* h, const void* kv, uint64_t kv_tokens, const float* noise, uint32_t n_steps,
                          const float* out, const float* states) {
  if (!h) return fail(PHYAI_ERR_INVALID_ARG, "handle is NULL");
  if (!noise || !out) return fail(PHYAI_ERR_INVALID_ARG, "noise / out_actions is NULL");
  if (n_steps == 0 || n_steps > 1000) return fail(PHYAI_ERR_INVALID_ARG, "n_steps must be in 1..1000");
  if (kv_tokens > 0 && !kv) return fail(PHYAI_ERR_INVALID_ARG, "prefix_kv is NULL with kv_tokens > 0");
  if (kv && !aligned16(kv)) return fail(PHYAI_ERR_INVALID_ARG, "prefix_kv must be 16-byte aligned");
  if ((reinterpret_cast<uintptr_t>(noise) & 3u) || (reinterpret_cast<uintptr_t>(out) & 3u))
    return fail(PHYAI_ERR_INVALID_ARG, "noise / out_actions must be 4-byte aligned");
  if (h->cfg.has_state_token && !states) return fail(PHYAI_ERR_INVALID_ARG, "state is NULL but the expert has a state token");
  return PHYAI_OK;
}

}  // namespace

// =============================================================================================
// C ABI
// =============================================================================================
extern "C" {

const char* phyai_last_error(void) { return g_err; }
const char* phyai_version(void) { return "phyai-b200 0.1 (sm_100a)"; }

size_t phyai_prefix_kv_bytes(const phyai_expert_config_t* c, uint64_t tokens) {
  if (!c || !c->n_layers || !c->n_kv_heads || !c->head_dim) return 0;
  return (size_t)c->n_layers * 2 * tokens * c->n_kv_heads * c->head_dim * kv_elem_bytes(c->dtype);
}

phyai_status_t phyai_expert_create(const phyai_expert_config_t* cfg, const phyai_weights_t* w, void* stream,
                                   phyai_expert_t** out) {
  if (!out) return fail(PHYAI_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  ST(check_config(cfg));
  if (!w) return fail(PHYAI_ERR_INVALID_ARG, "weights is NULL");
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0)
    return fail(PHYAI_ERR_CUDA, "no CUDA device: this library has no CPU fallback");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

  const bool ada = cfg->cond == PHYAI_COND_PI05_ADARMS;
  const bool tc = cfg->dtype != PHYAI_F32 && cfg->engine != PHYAI_ENGINE_SIMT;
  if (tc && !tc_shape_ok(cfg))
    return fail(PHYAI_ERR_UNSUPPORTED, "tensor path needs width, mlp_dim, q and qkv widths to be multiples of 128");
  // required pointers
  const bool need_state = cfg->has_state_token != 0;
  if (!w->action_in_w || !w->action_in_b || !w->time_mlp1_w || !w->time_mlp1_b || !w->time_mlp2_w || !w->time_mlp2_b ||
      !w->action_out_w || !w->action_out_b || !w->final_norm || (ada && !w->final_norm_b) ||
      (need_state && (!w->state_w || !w->state_b)) || !w->wq || !w->wk || !w->wv || !w->wo || !w->wgate || !w->wup ||
      !w->wdown || !w->norm1 || !w->norm2 || (ada && (!w->norm1_b || !w->norm2_b)))
    return fail(PHYAI_ERR_INVALID_ARG, "a required weight pointer is NULL");
  for (uint32_t l = 0; l < cfg->n_layers; ++l)
    if (!w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->wgate[l] || !w->wup[l] || !w->wdown[l] || !w->norm1[l] ||
        !w->norm2[l] || (ada && (!w->norm1_b[l] || !w->norm2_b[l])))
      return fail(PHYAI_ERR_INVALID_ARG, "a per-layer weight pointer is NULL (layer %u)", l);
  const bool a8 = cfg->dtype == PHYAI_W8A8_E4M3;     // e4m3 activations as well: the FP8 tensor path
  const bool w4 = cfg->dtype == PHYAI_W4A16;        // int4 codes + scales, expanded to bf16 images at create
  if (w4 && ((cfg->n_q_heads * cfg->head_dim) % 2 || (cfg->n_kv_heads * cfg->head_dim) % 2 || cfg->width % 2 || cfg->mlp_dim % 2))
    return fail(PHYAI_ERR_INVALID_ARG, "PHYAI_W4A16 stores two output channels per byte: output widths must be even");
  const bool w8 = cfg->dtype == PHYAI_W8E4M3_A16 || a8 || w4;   // per-output-channel scales
  if (a8 && !tc) return fail(PHYAI_ERR_UNSUPPORTED, "PHYAI_W8A8_E4M3 runs on the tensor path only (engine AUTO)");
  if (a8 && (cfg->width % 128 || cfg->mlp_dim % 128 || (cfg->n_q_heads * cfg->head_dim) % 128 || cfg->mlp_dim > 4096 ||
             cfg->width > 4096 || cfg->n_q_heads * cfg->head_dim > 4096))
    return fail(PHYAI_ERR_UNSUPPORTED, "PHYAI_W8A8_E4M3 needs contraction lengths that are multiples of 128 and at most 4096");
  if (w8)
    for (int m = 0; m < 7; ++m) {
      if (!w->scales[m]) return fail(PHYAI_ERR_INVALID_ARG, "scales[%d] is NULL", m);
      for (uint32_t l = 0; l < cfg->n_layers; ++l)
        if (!w->scales[m][l]) return fail(PHYAI_ERR_INVALID_ARG, "scales[%d][%u] is NULL", m, l);
    }

  phyai_expert* h = new (std::nothrow) phyai_expert();
  if (!h) return fail(PHYAI_ERR_OOM, "host allocation failed");
  h->cfg = *cfg;
  h->tc = tc, h->ada = ada, h->a8 = a8;
  Dims& d = h->d;
  d.L = cfg->n_layers, d.D = cfg->width, d.F = cfg->mlp_dim, d.Hq = cfg->n_q_heads, d.Hkv = cfg->n_kv_heads;
  d.dh = cfg->head_dim, d.Ds = cfg->state_dim, d.A = cfg->action_dim, d.H = cfg->horizon, d.ns = cfg->has_state_token;
  d.S = d.H + d.ns, d.Nq = d.Hq * d.dh, d.Nqkv = (d.Hq + 2 * d.Hkv) * d.dh;
  d.eps = cfg->rms_eps, d.gelu_exact = cfg->gelu_exact, d.block_causal = cfg->suffix_block_causal;
  h->sites = 2 * d.L + 1;
  h->Mpad = (int)(((size_t)cfg->max_batch * d.S + 255) / 256 * 256);
  const int D = d.D, L = d.L, kind = kind_of(cfg->dtype);     // storage of non-quantised tensors
  const int big_kind = w4 ? 3 : (w8 ? 2 : kind);              // storage of the seven big matrices
  const size_t Mp = h->Mpad;

  auto body = [&]() -> phyai_status_t {
    if (tc) CU(tc_gemm_setup());
    if (tc) CU(persist_gemm_setup());
    {
      int dev = 0;
      CU(cudaGetDevice(&dev));
      CU(cudaDeviceGetAttribute(&h->n_sm, cudaDevAttrMultiProcessorCount, dev));
    }
    CU(cudaStreamCreateWithFlags(&h->cap_stream, cudaStreamNonBlocking));
    ST(h->alloc(&h->status, 1, true));
    ST(h->alloc(&h->cu_internal, 2, true));
    if (tc) ST(h->alloc(&h->slab, (size_t)MAX_SLABS * 64 * D, true));
    ST(h->alloc(&h->order, (size_t)cfg->max_batch, true));
    ST(h->alloc(&h->rq, 1, true));
    // ---- small tensors -> fp32 ----
    if (need_state) {
      ST(h->alloc(&h->state_w, (size_t)d.Ds * D));
      ST(h->alloc(&h->state_b, D));
      launch_to_f32(w->state_w, kind, h->state_w, (size_t)d.Ds * D, st);
      launch_to_f32(w->state_b, kind, h->state_b, D, st);
    }
    ST(h->alloc(&h->Wout, (size_t)D * d.A));
    ST(h->alloc(&h->bout, d.A));
    launch_to_f32(w->action_out_w, kind, h->Wout, (size_t)D * d.A, st);
    launch_to_f32(w->action_out_b, kind, h->bout, d.A, st);
    ST(h->alloc(&h->b1, D));
    ST(h->alloc(&h->b2, D));
    launch_to_f32(w->time_mlp1_b, kind, h->b1, D, st);
    launch_to_f32(w->time_mlp2_b, kind, h->b2, D, st);
    ST(h->alloc(&h->Wc, (size_t)d.A * D));
    ST(h->alloc(&h->bcfold, D));
    ST(h->alloc(&h->W1tau, (size_t)D * D));
    float *Wa = nullptr, *ba = nullptr;
    ST(h->alloc(&Wa, (size_t)d.A * D));
    ST(h->alloc(&ba, D));
    launch_to_f32(w->action_in_w, kind, Wa, (size_t)d.A * D, st);
    launch_to_f32(w->action_in_b, kind, ba, D, st);
    const size_t esz = kind == 0 ? 4 : 2;
    if (!ada) {
      // fold the action projection into the first MLP layer: Wc = Wa W1[0:D], bcfold = ba W1[0:D] + b1
      launch_rows_gemm(Wa, D, w->time_mlp1_w, kind, 0, D, D, nullptr, nullptr, 0, h->Wc, D, d.A, st);
      launch_rows_gemm(ba, D, w->time_mlp1_w, kind, 0, D, D, h->b1, nullptr, 0, h->bcfold, D, 1, st);
      launch_to_f32(reinterpret_cast<const uint8_t*>(w->time_mlp1_w) + (size_t)D * D * esz, kind, h->W1tau,
                    (size_t)D * D, st);
      if (tc) {
        ST(h->alloc(&h->W2p, (size_t)D * D));
        launch_pack_tiled(w->time_mlp2_w, kind, h->W2p, D, D, 0, st);
      } else {
        ST(h->alloc(&h->W2f, (size_t)D * D));
        launch_to_f32(w->time_mlp2_w, kind, h->W2f, (size_t)D * D, st);
      }
    } else {
      CU(cudaMemcpyAsync(h->Wc, Wa, (size_t)d.A * D * 4, cudaMemcpyDeviceToDevice, st));
      CU(cudaMemcpyAsync(h->bcfold, ba, (size_t)D * 4, cudaMemcpyDeviceToDevice, st));
      launch_to_f32(w->time_mlp1_w, kind, h->W1tau, (size_t)D * D, st);
      ST(h->alloc(&h->W2f, (size_t)D * D));
      launch_to_f32(w->time_mlp2_w, kind, h->W2f, (size_t)D * D, st);
    }
    // ---- norm parameters ----
    if (!ada) {
      ST(h->alloc(&h->gains, (size_t)h->sites * D));
      float* tmp = nullptr;
      ST(h->alloc(&tmp, D));
      for (int s = 0; s < h->sites; ++s) {
        const void* src = s == 2 * L ? w->final_norm : (s & 1 ? w->norm2[s / 2] : w->norm1[s / 2]);
        launch_to_f32(src, kind, tmp, D, st);
        launch_one_plus(tmp, h->gains + (size_t)s * D, D, st);
      }
    } else {
      h->wmod_kind = kind;
      const size_t wsite = (size_t)D * 3 * D * esz;
      uint8_t* wm = nullptr;
      ST(h->alloc(&wm, wsite * h->sites));
      h->wmod = wm;
      ST(h->alloc(&h->bmod, (size_t)h->sites * 3 * D));
      for (int s = 0; s < h->sites; ++s) {
        const void* src = s == 2 * L ? w->final_norm : (s & 1 ? w->norm2[s / 2] : w->norm1[s / 2]);
        const void* bsrc = s == 2 * L ? w->final_norm_b : (s & 1 ? w->norm2_b[s / 2] : w->norm1_b[s / 2]);
        CU(cudaMemcpyAsync(wm + s * wsite, src, wsite, cudaMemcpyDeviceToDevice, st));
        launch_to_f32(bsrc, kind, h->bmod + (size_t)s * 3 * D, (size_t)3 * D, st);
      }
    }
    // ---- the seven big matrices per layer ----
    const int Nq = d.Nq, Nkv = d.Hkv * d.dh, Nqkv = d.Nqkv, F = d.F;
    __nv_bfloat16 *pq_all = nullptr, *po_all = nullptr, *pg_all = nullptr, *pu_all = nullptr, *pd_all = nullptr;
    if (tc) {   // one allocation per matrix kind, layers at a fixed stride (the persistent kernel indexes by layer)
      ST(h->alloc(&pq_all, (size_t)L * D * Nqkv)); ST(h->alloc(&po_all, (size_t)L * Nq * D));
      ST(h->alloc(&pg_all, (size_t)L * D * F)); ST(h->alloc(&pu_all, (size_t)L * D * F));
      ST(h->alloc(&pd_all, (size_t)L * F * D));
      h->il_ok = F % 64 == 0 && !a8;   // (W8A8 keeps to the general kernels: no interleaved image, no cluster path)
      if (h->il_ok) ST(h->alloc(&h->p_gu_all, (size_t)L * D * 2 * F));
      // token counts that use 256-token tiles: the persistent gate / up kernel and its weight image
      if (pick_nt((int)(cfg->max_batch * d.S)) == 256 && persist_gemm_supported((int)(cfg->max_batch * d.S), 2 * F, D, h->Mpad, a8)) {
        ST(h->alloc(&h->p_gu16, (size_t)L * D * 2 * F / (a8 ? 2 : 1)));
        if ((d.dh == 128 || d.dh == 256) && d.S <= 64) ST(h->alloc(&h->p_qkv16, (size_t)L * D * Nqkv / (a8 ? 2 : 1)));
      }
      // cluster split-K path (one 64-token tile): every projection must fit the kernel's resident stages
      auto fits = [&](int N, int K, bool qkv) {
        return b1_gemm_supported(N, K, b1_pick_cluster(N / 128, K / 64, h->n_sm), h->n_sm, qkv);
      };
      h->b1_ok = h->il_ok && (d.dh == 128 || d.dh == 256) && D % 128 == 0 && d.S <= 64 && fits(Nqkv, D, true) &&
                 fits(D, Nq, false) && fits(2 * F, D, false) && fits(D, F, false);
      if (w8) {
        ST(h->alloc(&h->s_qkv_all, (size_t)L * Nqkv)); ST(h->alloc(&h->s_o_all, (size_t)L * D));
        ST(h->alloc(&h->s_g_all, (size_t)L * F)); ST(h->alloc(&h->s_u_all, (size_t)L * F));
        ST(h->alloc(&h->s_d_all, (size_t)L * D));
      }
    }
    for (int l = 0; l < L; ++l) {
      const float* sq = w8 ? w->scales[0][l] : nullptr; const float* sk = w8 ? w->scales[1][l] : nullptr;
      const float* sv = w8 ? w->scales[2][l] : nullptr; const float* so = w8 ? w->scales[3][l] : nullptr;
      const float* sg = w8 ? w->scales[4][l] : nullptr; const float* su = w8 ? w->scales[5][l] : nullptr;
      const float* sd = w8 ? w->scales[6][l] : nullptr;
      if (tc) {
        __nv_bfloat16 *pq = pq_all + (size_t)l * D * Nqkv, *po = po_all + (size_t)l * Nq * D;
        __nv_bfloat16 *pg = pg_all + (size_t)l * D * F, *pu = pu_all + (size_t)l * D * F, *pd = pd_all + (size_t)l * F * D;
        if (h->p_gu16) {
          // (bf16 image: 2 bytes per weight; W8A8: the e4m3 codes, 1 byte per weight, in the first half of the layer's slot)
          __nv_bfloat16* p16 = h->p_gu16 + (size_t)l * D * 2 * F / (a8 ? 2 : 1);
          if (a8) {
            launch_pack_bytes(reinterpret_cast<const uint8_t*>(w->wgate[l]), reinterpret_cast<uint8_t*>(p16), D, F, 0, st, 16, 0, 0, 1);
            launch_pack_bytes(reinterpret_cast<const uint8_t*>(w->wup[l]), reinterpret_cast<uint8_t*>(p16), D, F, 0, st, 16, 1, 0, 1);
          } else {
            launch_pack_tiled(w->wgate[l], big_kind, p16, D, F, 0, st, 16, 0);
            launch_pack_tiled(w->wup[l], big_kind, p16, D, F, 0, st, 16, 1);
          }
        }
        if (h->p_qkv16) {
          __nv_bfloat16* p16 = h->p_qkv16 + (size_t)l * D * Nqkv / (a8 ? 2 : 1);
          if (a8) {
            auto u8 = [](const void* p) { return reinterpret_cast<const uint8_t*>(p); };
            uint8_t* o8 = reinterpret_cast<uint8_t*>(p16);
            launch_pack_bytes(u8(w->wq[l]), o8, D, Nq, 0, st, 0, 0, d.dh, 1, 1);
            launch_pack_bytes(u8(w->wk[l]), o8, D, Nkv, Nq, st, 0, 0, d.dh, 1, 1);
            launch_pack_bytes(u8(w->wv[l]), o8, D, Nkv, Nq + Nkv, st, 0, 0, 0, 1, 1);
          } else {
            launch_pack_tiled(w->wq[l], big_kind, p16, D, Nq, 0, st, 0, 0, d.dh, 1);
            launch_pack_tiled(w->wk[l], big_kind, p16, D, Nkv, Nq, st, 0, 0, d.dh, 1);
            launch_pack_tiled(w->wv[l], big_kind, p16, D, Nkv, Nq + Nkv, st, 0, 0, 0, 1);
          }
        }
        if (h->il_ok) {
          __nv_bfloat16* pgu = h->p_gu_all + (size_t)l * D * 2 * F;
          launch_pack_tiled(w->wgate[l], big_kind, pgu, D, F, 0, st, 64, 0);
          launch_pack_tiled(w->wup[l], big_kind, pgu, D, F, 0, st, 64, 1);
        }
        if (a8) {
          // the e4m3 codes themselves as operand images: blocks of 128 channels x 128 k (the allocations are sized
          // for bf16 images: half of each is used)
          auto u8 = [](const void* p) { return reinterpret_cast<const uint8_t*>(p); };
          auto o8 = [](__nv_bfloat16* p) { return reinterpret_cast<uint8_t*>(p); };
          launch_pack_bytes(u8(w->wq[l]), o8(pq), D, Nq, 0, st, 0, 0, d.dh, 1);
          launch_pack_bytes(u8(w->wk[l]), o8(pq), D, Nkv, Nq, st, 0, 0, d.dh, 1);
          launch_pack_bytes(u8(w->wv[l]), o8(pq), D, Nkv, Nq + Nkv, st, 0, 0, 0, 1);
          launch_pack_bytes(u8(w->wo[l]), o8(po), Nq, D, 0, st, 0, 0, 0, 1);
          launch_pack_bytes(u8(w->wgate[l]), o8(pg), D, F, 0, st, 0, 0, 0, 1);
          launch_pack_bytes(u8(w->wup[l]), o8(pu), D, F, 0, st, 0, 0, 0, 1);
          launch_pack_bytes(u8(w->wdown[l]), o8(pd), F, D, 0, st, 0, 0, 0, 1);
        } else {
          launch_pack_tiled(w->wq[l], big_kind, pq, D, Nq, 0, st, 0, 0, d.dh);
          launch_pack_tiled(w->wk[l], big_kind, pq, D, Nkv, Nq, st, 0, 0, d.dh);
          launch_pack_tiled(w->wv[l], big_kind, pq, D, Nkv, Nq + Nkv, st);
          launch_pack_tiled(w->wo[l], big_kind, po, Nq, D, 0, st);
          launch_pack_tiled(w->wgate[l], big_kind, pg, D, F, 0, st);
          launch_pack_tiled(w->wup[l], big_kind, pu, D, F, 0, st);
          launch_pack_tiled(w->wdown[l], big_kind, pd, F, D, 0, st);
        }
        h->p_qkv.push_back(pq), h->p_o.push_back(po), h->p_g.push_back(pg), h->p_u.push_back(pu), h->p_d.push_back(pd);
        if (w8 && !a8 && h->b1_ok) {
          // one byte per weight for the single-tile (HBM-bound) path; larger batches are tensor-bound and keep using
          // the bf16 images above
          uint8_t *bq, *bo, *bgu, *bd;
          const size_t div = w4 ? 2 : 1;     // int4: half a byte per weight
          ST(h->alloc(&bq, (size_t)D * Nqkv / div)); ST(h->alloc(&bo, (size_t)Nq * D / div));
          ST(h->alloc(&bgu, (size_t)D * 2 * F / div)); ST(h->alloc(&bd, (size_t)F * D / div));
          auto pack = [&](const void* src, uint8_t* dst, int K, int N, int n_off, int il = 0, int second = 0, int perm = 0) {
            if (w4) launch_pack_nibbles(reinterpret_cast<const uint8_t*>(src), dst, K, N, n_off, st, il, second, perm);
            else launch_pack_bytes(reinterpret_cast<const uint8_t*>(src), dst, K, N, n_off, st, il, second, perm);
          };
          pack(w->wq[l], bq, D, Nq, 0, 0, 0, d.dh);
          pack(w->wk[l], bq, D, Nkv, Nq, 0, 0, d.dh);
          pack(w->wv[l], bq, D, Nkv, Nq + Nkv);
          pack(w->wo[l], bo, Nq, D, 0);
          pack(w->wgate[l], bgu, D, F, 0, 64, 0);
          pack(w->wup[l], bgu, D, F, 0, 64, 1);
          pack(w->wdown[l], bd, F, D, 0);
          h->b_qkv.push_back(bq), h->b_o.push_back(bo), h->b_gu.push_back(bgu), h->b_d.push_back(bd);
        }
        float *cq = nullptr, *co = nullptr, *cg = nullptr, *cu = nullptr, *cd = nullptr;
        if (w8) {
          cq = h->s_qkv_all + (size_t)l * Nqkv, co = h->s_o_all + (size_t)l * D, cg = h->s_g_all + (size_t)l * F;
          cu = h->s_u_all + (size_t)l * F, cd = h->s_d_all + (size_t)l * D;
          launch_permute_scales(sq, cq, Nq, 0, d.dh, st);
          launch_permute_scales(sk, cq, Nkv, Nq, d.dh, st);
          CU(cudaMemcpyAsync(cq + Nq + Nkv, sv, (size_t)Nkv * 4, cudaMemcpyDeviceToDevice, st));
          CU(cudaMemcpyAsync(co, so, (size_t)D * 4, cudaMemcpyDeviceToDevice, st));
          CU(cudaMemcpyAsync(cg, sg, (size_t)F * 4, cudaMemcpyDeviceToDevice, st));
          CU(cudaMemcpyAsync(cu, su, (size_t)F * 4, cudaMemcpyDeviceToDevice, st));
          CU(cudaMemcpyAsync(cd, sd, (size_t)D * 4, cudaMemcpyDeviceToDevice, st));
        }
        h->s_qkv.push_back(cq), h->s_o.push_back(co), h->s_g.push_back(cg), h->s_u.push_back(cu), h->s_d.push_back(cd);
      } else {
        float *fq, *fo, *fg, *fu, *fd;
        ST(h->alloc(&fq, (size_t)D * Nqkv)); ST(h->alloc(&fo, (size_t)Nq * D));
        ST(h->alloc(&fg, (size_t)D * F)); ST(h->alloc(&fu, (size_t)D * F)); ST(h->alloc(&fd, (size_t)F * D));
        launch_copy_cols(w->wq[l], big_kind, sq, fq, D, Nq, Nqkv, 0, st);
        launch_copy_cols(w->wk[l], big_kind, sk, fq, D, Nkv, Nqkv, Nq, st);
        launch_copy_cols(w->wv[l], big_kind, sv, fq, D, Nkv, Nqkv, Nq + Nkv, st);
        launch_copy_cols(w->wo[l], big_kind, so, fo, Nq, D, D, 0, st);
        launch_copy_cols(w->wgate[l], big_kind, sg, fg, D, F, F, 0, st);
        launch_copy_cols(w->wup[l], big_kind, su, fu, D, F, F, 0, st);
        launch_copy_cols(w->wdown[l], big_kind, sd, fd, F, D, D, 0, st);
        h->f_qkv.push_back(fq), h->f_o.push_back(fo), h->f_g.push_back(fg), h->f_u.push_back(fu), h->f_d.push_back(fd);
      }
    }
    // ---- rotary table ----
    if (cfg->rope_theta > 0.f) {
      const int npos = (int)cfg->max_prefix_len + d.S;
      ST(h->alloc(&h->rope, (size_t)npos * (d.dh / 2)));
      launch_rope_table(h->rope, npos, d.dh, (double)cfg->rope_theta, st);
    }
    // ---- workspace (zeroed: padding rows of the tiled buffers stay finite) ----
    ST(h->alloc(&h->h, Mp * D, true));
    ST(h->alloc(&h->qkv, Mp * Nqkv, true));
    if (tc && (d.dh == 128 || d.dh == 256)) {   // rotated bf16 q / k / v for the tcgen05 and cluster attention kernels
      ST(h->alloc(&h->qr_big, Mp * d.Nq, true));
      ST(h->alloc(&h->kr_big, Mp * (size_t)(d.Hkv * d.dh), true));
      ST(h->alloc(&h->vr_big, Mp * (size_t)(d.Hkv * d.dh), true));
    }
    ST(h->alloc(&h->state_tok, (size_t)cfg->max_batch * D, true));
    if (a8) {   // tiled e4m3 activations of the widest projection input, and the per-token scales
      const size_t kmax = (size_t)std::max(std::max(D, d.Nq), d.F);
      ST(h->alloc(&h->xq, Mp * kmax, true));
      ST(h->alloc(&h->xs, Mp, true));
    }
    if (tc) {
      h->attn_mma = attention_mma_supported(d);
      if (h->attn_mma) {
        size_t need = 0;
        for (int bb = 1; bb <= (int)cfg->max_batch; ++bb) {
          const size_t n = attention_scratch_floats(d, bb, attention_pick_splits(d, bb, (int)cfg->max_prefix_len));
          need = n > need ? n : need;
          if (attention_tc_supported(d)) {
            const size_t n2 = attention_scratch_floats(d, bb, attention_tc_splits(d, bb, h->n_sm, (int)cfg->max_prefix_len));
            need = n2 > need ? n2 : need;
          }
        }
        if (need) ST(h->alloc(&h->attn_scratch, need, true));
      }
      // cluster split-K path (one 64-token tile): compact 64-row activation tiles and the norm partials
      if (h->b1_ok) {
        ST(h->alloc(&h->xn64, (size_t)64 * D, true));
        ST(h->alloc(&h->attn64, (size_t)64 * Nq, true));
        ST(h->alloc(&h->m64, (size_t)64 * F, true));
        ST(h->alloc(&h->ss_a, (size_t)(D / 128) * 64, true));
        ST(h->alloc(&h->ss_b, (size_t)(D / 128) * 64, true));
        if (attention_b1_supported(d) && d.Hq >= 2)   // q as operand tiles of the cluster attention kernel: up to 64 query rows
          ST(h->alloc(&h->q_tiles, (size_t)64 * (d.Hq / 2) * 128 * d.dh, true));
        if (d.block_causal && d.ns && !ada) {
          // per-layer suffix K / V (key row 0 = the cached state token) for as many requests as fit one 64-token tile
          const size_t per_layer = (size_t)(64 / d.S > 0 ? 64 / d.S : 1) * d.Hkv * d.S * d.dh;
          ST(h->alloc(&h->kr_st, (size_t)L * per_layer, true));
          ST(h->alloc(&h->vr_st, (size_t)L * per_layer, true));
        }
      }
      ST(h->alloc(&h->xn_t, Mp * D, true));
      ST(h->alloc(&h->attn_t, Mp * Nq, true));
      ST(h->alloc(&h->m_t, Mp * F, true));
      if (!ada) ST(h->alloc(&h->u_t, Mp * D, true));
    } else {
      ST(h->alloc(&h->xn_f, Mp * D, true));
      ST(h->alloc(&h->attn_f, Mp * Nq, true));
      ST(h->alloc(&h->m_f, Mp * F, true));
      if (!ada) ST(h->alloc(&h->u_f, Mp * D, true));
    }
    CU(cudaGetLastError());
    CU(cudaStreamSynchronize(st));
    CU(cudaDeviceSynchronize());  // the zero-fills above ran on the default stream
    return PHYAI_OK;
  };
  phyai_status_t s = body();
  if (s != PHYAI_OK) {
    char keep[sizeof(g_err)];
    memcpy(keep, g_err, sizeof(keep));
    phyai_expert_destroy(h);
    memcpy(g_err, keep, sizeof(keep));
    return s;
  }
  *out = h;
  return PHYAI_OK;
}

void phyai_expert_destroy(phyai_expert_t* h) {
  if (!h) return;
  cudaDeviceSynchronize();
  for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
  if (h->cap_stream) cudaStreamDestroy(h->cap_stream);
  for (void* p : h->allocs) cudaFree(p);
  delete h;
}

phyai_status_t phyai_denoise(phyai_expert_t* h, const void* prefix_kv, uint64_t kv_tokens, uint32_t prefix_len,
                             const float* state, const float* noise, uint32_t n_steps, float* out, void* stream) {
  ST(check_call(h, prefix_kv, kv_tokens, noise, n_steps, out, state));
  if (prefix_len > h->cfg.max_prefix_len || prefix_len > kv_tokens)
    return fail(PHYAI_ERR_INVALID_ARG, "prefix_len %u exceeds max_prefix_len %u or kv_tokens %llu", prefix_len,
                h->cfg.max_prefix_len, (unsigned long long)kv_tokens);
  Request r{};
  r.prefix_kv = prefix_kv, r.kv_tokens = kv_tokens, r.cu_lens = nullptr, r.states = state, r.noise = noise, r.x = out;
  r.batch = 1, r.single_len = (int)prefix_len;
  return run(h, r, (int)n_steps, reinterpret_cast<cudaStream_t>(stream));
}

phyai_status_t phyai_denoise_batched(phyai_expert_t* h, uint32_t batch, const void* prefix_kv, uint64_t kv_tokens,
                                     const int32_t* cu, const float* states, const float* noise, uint32_t n_steps,
                                     float* out, void* stream) {
  ST(check_call(h, prefix_kv, kv_tokens, noise, n_steps, out, states));
  if (batch == 0 || batch > h->cfg.max_batch)
    return fail(PHYAI_ERR_INVALID_ARG, "batch %u outside 1..max_batch (%u)", batch, h->cfg.max_batch);
  if (!cu) return fail(PHYAI_ERR_INVALID_ARG, "cu_prefix_lens is NULL");
  if (kv_tokens > (uint64_t)INT32_MAX) return fail(PHYAI_ERR_INVALID_ARG, "kv_tokens exceeds int32 range");
  Request r{};
  r.prefix_kv = prefix_kv, r.kv_tokens = kv_tokens, r.cu_lens = cu, r.states = states, r.noise = noise, r.x = out;
  r.batch = (int)batch, r.single_len = 0;
  return run(h, r, (int)n_steps, reinterpret_cast<cudaStream_t>(stream));
}

static phyai_status_t ensure_staging(phyai_expert* h) {
  if (h->stg_noise) return PHYAI_OK;
  const size_t B = h->cfg.max_batch;
  h->stg_kv_bytes = phyai_prefix_kv_bytes(&h->cfg, (uint64_t)B * h->cfg.max_prefix_len);
  uint8_t* kv = nullptr;
  ST(h->alloc(&kv, h->stg_kv_bytes));
  h->stg_kv = kv;
  ST(h->alloc(&h->stg_states, B * (h->d.Ds ? h->d.Ds : 1)));
  ST(h->alloc(&h->stg_out, B * h->d.H * h->d.A));
  ST(h->alloc(&h->stg_cu, B + 1));
  ST(h->alloc(&h->stg_noise, B * h->d.H * h->d.A));
  return PHYAI_OK;
}

phyai_status_t phyai_denoise_batched_host(phyai_expert_t* h, uint32_t batch, const void* prefix_kv, uint64_t kv_tokens,
                                          const int32_t* cu, const float* states, const float* noise, uint32_t n_steps,
                                          float* out, void* stream) {
  ST(check_call(h, prefix_kv, kv_tokens, noise, n_steps, out, states));
  if (batch == 0 || batch > h->cfg.max_batch)
    return fail(PHYAI_ERR_INVALID_ARG, "batch %u outside 1..max_batch (%u)", batch, h->cfg.max_batch);
  if (!cu) return fail(PHYAI_ERR_INVALID_ARG, "cu_prefix_lens is NULL");
  if (kv_tokens > (uint64_t)h->cfg.max_batch * h->cfg.max_prefix_len)
    return fail(PHYAI_ERR_INVALID_ARG, "kv_tokens exceeds the staging capacity max_batch * max_prefix_len");
  ST(ensure_staging(h));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const size_t kvb = phyai_prefix_kv_bytes(&h->cfg, kv_tokens), ha = (size_t)batch * h->d.H * h->d.A * 4;
  if (kvb) CU(cudaMemcpyAsync(h->stg_kv, prefix_kv, kvb, cudaMemcpyHostToDevice, st));
  CU(cudaMemcpyAsync(h->stg_cu, cu, (size_t)(batch + 1) * 4, cudaMemcpyHostToDevice, st));
  if (states) CU(cudaMemcpyAsync(h->stg_states, states, (size_t)batch * h->d.Ds * 4, cudaMemcpyHostToDevice, st));
  CU(cudaMemcpyAsync(h->stg_noise, noise, ha, cudaMemcpyHostToDevice, st));
  Request r{};
  r.prefix_kv = h->stg_kv, r.kv_tokens = kv_tokens, r.cu_lens = h->stg_cu, r.states = states ? h->stg_states : nullptr;
  r.noise = h->stg_noise, r.x = h->stg_out, r.batch = (int)batch, r.single_len = 0;
  ST(run(h, r, (int)n_steps, st));
  CU(cudaMemcpyAsync(out, h->stg_out, ha, cudaMemcpyDeviceToHost, st));
  return PHYAI_OK;
}

phyai_status_t phyai_denoise_host(phyai_expert_t* h, const void* prefix_kv, uint64_t kv_tokens, uint32_t prefix_len,
                                  const float* state, const float* noise, uint32_t n_steps, float* out, void* stream) {
  if (!h) return fail(PHYAI_ERR_INVALID_ARG, "handle is NULL");
  if (prefix_len > h->cfg.max_prefix_len || prefix_len > kv_tokens)
    return fail(PHYAI_ERR_INVALID_ARG, "prefix_len %u exceeds max_prefix_len %u or kv_tokens %llu", prefix_len,
                h->cfg.max_prefix_len, (unsigned long long)kv_tokens);
  ST(check_call(h, prefix_kv, kv_tokens, noise, n_steps, out, state));
  ST(ensure_staging(h));
  if (kv_tokens > (uint64_t)h->cfg.max_batch * h->cfg.max_prefix_len)
    return fail(PHYAI_ERR_INVALID_ARG, "kv_tokens exceeds the staging capacity max_batch * max_prefix_len");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const size_t kvb = phyai_prefix_kv_bytes(&h->cfg, kv_tokens), ha = (size_t)h->d.H * h->d.A * 4;
  if (kvb) CU(cudaMemcpyAsync(h->stg_kv, prefix_kv, kvb, cudaMemcpyHostToDevice, st));
  if (state) CU(cudaMemcpyAsync(h->stg_states, state, (size_t)h->d.Ds * 4, cudaMemcpyHostToDevice, st));
  CU(cudaMemcpyAsync(h->stg_noise, noise, ha, cudaMemcpyHostToDevice, st));
  Request r{};
  r.prefix_kv = h->stg_kv, r.kv_tokens = kv_tokens, r.cu_lens = nullptr, r.states = state ? h->stg_states : nullptr;
  r.noise = h->stg_noise, r.x = h->stg_out, r.batch = 1, r.single_len = (int)prefix_len;
  ST(run(h, r, (int)n_steps, st));
  CU(cudaMemcpyAsync(out, h->stg_out, ha, cudaMemcpyDeviceToHost, st));
  return PHYAI_OK;
}

phyai_status_t phyai_poll_status(phyai_expert_t* h) {
  if (!h) return fail(PHYAI_ERR_INVALID_ARG, "handle is NULL");
  int v = 0;
  CU(cudaMemcpy(&v, h->status, sizeof(int), cudaMemcpyDeviceToHost));
  if (v != 0) {
    CU(cudaMemset(h->status, 0, sizeof(int)));
    if (v == ST_TIMEOUT) return fail(PHYAI_ERR_TIMEOUT, "a bounded device-side wait expired; results are invalid");
    return fail(PHYAI_ERR_INVALID_ARG, "device-side validation of cu_prefix_lens failed; nothing was written");
  }
  return PHYAI_OK;
}

phyai_status_t phyai_set_option(phyai_expert_t* h, const char* key, int64_t value) {
  if (!h || !key) return fail(PHYAI_ERR_INVALID_ARG, "handle or key is NULL");
  if (!strcmp(key, "use_graph")) {
    h->use_graph = value != 0;
    return PHYAI_OK;
  }
  if (!strcmp(key, "use_tc_attention")) {
    h->use_tc_attention = value != 0;
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    return PHYAI_OK;
  }
  if (!strcmp(key, "slab_splits")) {
    if (value < 1 || value > MAX_SLABS) return fail(PHYAI_ERR_INVALID_ARG, "slab_splits out of range");
    h->slab_splits = (int)value;
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    return PHYAI_OK;
  }
  if (!strcmp(key, "use_fused_oproj")) {
    h->use_fused_oproj = value != 0;
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    return PHYAI_OK;
  }
  if (!strcmp(key, "use_cluster_attention")) {
    h->use_cluster_attention = value != 0;
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    return PHYAI_OK;
  }
  if (!strcmp(key, "b1_attn_hpc")) {
    if (value < 0 || value > 2) return fail(PHYAI_ERR_INVALID_ARG, "b1_attn_hpc is 0 (choose), 1 or 2");
    h->b1_attn_hpc = (int)value;
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    return PHYAI_OK;
  }
  if (!strcmp(key, "use_b1_step")) {
    h->use_b1_step = value != 0;
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    return PHYAI_OK;
  }
  if (!strcmp(key, "use_state_cache")) {
    h->use_state_cache = value != 0;
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    return PHYAI_OK;
  }
  if (!strcmp(key, "use_w8_inkernel")) {
    h->use_w8_inkernel = value != 0;
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    return PHYAI_OK;
  }
  if (!strcmp(key, "use_b1_attention")) {
    h->use_b1_attention = value != 0;
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    return PHYAI_OK;
  }
  if (!strcmp(key, "use_cluster_gemm") || !strcmp(key, "b1_c_qkv") || !strcmp(key, "b1_c_o") || !strcmp(key, "b1_c_gu") ||
      !strcmp(key, "b1_c_d")) {
    if (!strcmp(key, "use_cluster_gemm")) {
      h->use_cluster_gemm = value != 0;
    } else {
      if (value < 0 || value > 8) return fail(PHYAI_ERR_INVALID_ARG, "cluster size out of range 0..8");
      h->b1_c[!strcmp(key, "b1_c_qkv") ? 0 : !strcmp(key, "b1_c_o") ? 1 : !strcmp(key, "b1_c_gu") ? 2 : 3] = (int)value;
    }
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    return PHYAI_OK;
  }
  if (!strcmp(key, "trace")) {
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    if (value == 0) {
      h->trace = nullptr;      // (the buffer stays allocated until destroy)
      return PHYAI_OK;
    }
    if (!h->trace_buf) ST(h->alloc(&h->trace_buf, (size_t)TRACE_SLOTS * TRACE_STAMPS, true));
    h->trace = h->trace_buf;
    return PHYAI_OK;
  }
  if (!strcmp(key, "use_persistent_gu") || !strcmp(key, "use_persistent_qkv") || !strcmp(key, "use_attn_splits")) {
    (!strcmp(key, "use_persistent_gu") ? h->use_persistent_gu : !strcmp(key, "use_attn_splits") ? h->use_attn_splits : h->use_persistent_qkv) = value != 0;
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    return PHYAI_OK;
  }
  if (!strcmp(key, "trace_all_from")) {
    if (value < 0 || value >= TRACE_SLOTS) return fail(PHYAI_ERR_INVALID_ARG, "trace_all_from out of range");
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
    h->trace_all_from = (int)value;
    if (h->trace_buf) CU(cudaMemset(h->trace_buf, 0, (size_t)TRACE_SLOTS * TRACE_STAMPS * sizeof(unsigned long long)));
    return PHYAI_OK;
  }
  if (!strcmp(key, "wait_limit")) {
    if (value < 1 || value > (int64_t)0x7fffffff) return fail(PHYAI_ERR_INVALID_ARG, "wait_limit out of range");
    h->wait_limit = (unsigned)value;
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);  // the limit is baked into captured launches
    h->graphs.clear();
    return PHYAI_OK;
  }
  return fail(PHYAI_ERR_INVALID_ARG, "unknown option '%s'", key);
}

phyai_status_t phyai_read_trace(phyai_expert_t* h, uint64_t* out, size_t capacity, uint32_t* n_slots, uint32_t* n_stamps) {
  if (!h || !out || !n_slots || !n_stamps) return fail(PHYAI_ERR_INVALID_ARG, "NULL argument");
  if (!h->trace) return fail(PHYAI_ERR_INVALID_ARG, "tracing is off (phyai_set_option(h, \"trace\", 1))");
  const size_t n = (size_t)TRACE_SLOTS * TRACE_STAMPS;
  if (capacity < n) return fail(PHYAI_ERR_INVALID_ARG, "capacity %zu < %zu entries", capacity, n);
  CU(cudaMemcpy(out, h->trace, n * sizeof(uint64_t), cudaMemcpyDeviceToHost));
  *n_slots = TRACE_SLOTS, *n_stamps = TRACE_STAMPS;
  return PHYAI_OK;
}

uint64_t phyai_launches_per_call(phyai_expert_t* h, uint32_t batch, uint32_t n_steps) {
  if (!h) return 0;
  auto it = h->launch_counts.find(std::make_pair((int)batch, (int)n_steps));
  return it == h->launch_counts.end() ? 0 : it->second + 1 /* request-block kernel */;
}

}  // extern "C"
