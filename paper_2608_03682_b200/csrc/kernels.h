// Host-callable launchers of every kernel family.  Each launcher only enqueues on `st`.
#pragma once

#include "common.cuh"

#include <atomic>
#include <utility>

namespace phyai {

// cudaFuncSetAttribute acts on the current device, so "already configured" is remembered per device (bit d of the
// mask = device d; devices beyond 63 are configured on every launch).  Concurrent first launches may both
// configure, which is harmless.
struct PerDeviceOnce {
  std::atomic<unsigned long long> mask{0};
  int dev = -1;
  bool needed() {
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev > 63) {
      dev = -1;
      return true;
    }
    return !((mask.load(std::memory_order_acquire) >> dev) & 1ull);
  }
  void done() {
    if (dev >= 0) mask.fetch_or(1ull << dev, std::memory_order_release);
  }
};

// Launch with programmatic stream serialization (see pdl_enter in common.cuh): only for kernels that call
// pdl_enter() before touching global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid, cfg.blockDim = block, cfg.dynamicSmemBytes = smem, cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at, cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

struct Dims {
  int L, D, F, Hq, Hkv, dh, Ds, A, H, ns, S, Nqkv, Nq;
  float eps;
  int gelu_exact, block_causal;
  // Suffix keys of the cluster kernels when they differ from the query rows (state-token caching): a request's
  // rotated suffix K / V rows are Sk_stride rows apart per kv head, the first Sk of them exist, and query row i is
  // key row koff + i (position prefix_len + koff + i).  All zero = "same as the queries" (Sk = Sk_stride = S, koff = 0).
  int Sk, Sk_stride, koff;
};
inline int suffix_keys(const Dims& d) { return d.Sk > 0 ? d.Sk : d.S; }
inline int suffix_key_stride(const Dims& d) { return d.Sk_stride > 0 ? d.Sk_stride : d.S; }

// ---- request block ---------------------------------------------------------------------------
void launch_set_request(Request* dst, const Request& src, int* cu_internal, cudaStream_t st, int* order = nullptr);
void launch_validate(const Request* rq, int* status, int max_prefix, int* order, cudaStream_t st);

// ---- one-off table / packing kernels (CUDA cores, fp64 accumulation where cheap) ---------------
// src_kind: 0 = float32, 1 = bfloat16, 2 = e4m3 byte codes, 3 = int4 codes (two neighbouring elements of a row per
// byte, the even one in the low nibble; rows of even length)
void launch_to_f32(const void* src, int src_kind, float* dst, size_t n, cudaStream_t st);
// dst[r][col_off + c] = src[r][c] * (scale ? scale[c] : 1)
void launch_copy_cols(const void* src, int src_kind, const float* scale, float* dst, int rows, int cols, int ld_dst,
                      int col_off, cudaStream_t st);
// [in=K][out=N] source -> 128x64 blocks of the 128-byte-swizzled K-major bf16 image, out channel
// n stored at packed row n_off + n of a matrix with KC = K/64 column chunks.
// With il_group > 0 the channels of two matrices are interleaved in groups of il_group rows
// (il_second selects the second matrix): packed row = (n / g) * 2g + n % g + (second ? g : 0).
// With perm_dh > 0 the channels follow the rotary-pair row order of the fused QKV matrix
// (qkv_channel_to_packed).  With pair16 the rows of every 128-row tile are then interleaved in groups of 16: packed
// row r of the tile goes to row 32 ((r % 64) / 16) + 16 (r / 64) + r % 16 (rows r and r + 64 end up 16 apart).
void launch_pack_tiled(const void* src, int src_kind, __nv_bfloat16* dst, int K, int N, int n_off, cudaStream_t st,
                       int il_group = 0, int il_second = 0, int perm_dh = 0, int pair16 = 0);
// e4m3 codes [in=K][out=N] -> byte blocks [N/128][K/64][128][64] in the packed row order of launch_pack_tiled
void launch_pack_bytes(const uint8_t* src, uint8_t* dst, int K, int N, int n_off, cudaStream_t st, int il_group = 0,
                       int il_second = 0, int perm_dh = 0, int wide = 0, int pair16 = 0);
// (wide: blocks [N/128][K/128][128][128] instead, the 16-byte chunks of a row XOR-swizzled by row & 7: the e4m3
// operand image of the FP8 tensor path)
// row-major bf16 [M][K] (K a multiple of 8, 16-byte aligned rows) -> the tiled bf16 layout of the GEMM inputs
void launch_rows_to_tiled(const __nv_bfloat16* x, __nv_bfloat16* tiled, int M, int K, int rows_pad, cudaStream_t st);
// Per-token e4m3 quantization of a tiled bf16 activation matrix [K/64][rows_pad][64] (W8A8): scale[r] = max|x_r| / 448
// (1 for a zero row), codes = round-to-nearest-even e4m3 of x / scale, saturating, written as the tiled e4m3 matrix
// [K/128][rows_pad][128] with the same 16-byte chunk swizzle.  Rows >= M are left alone.
void launch_quant_rows(const int* status, const __nv_bfloat16* x, uint8_t* out, float* scale, int rows_pad, int M, int K,
                       cudaStream_t st);
// int4 codes [K][N/2] (two neighbouring out channels per byte) -> nibble blocks [N/128][K/64][128][32] in the packed
// row order of launch_pack_tiled, byte j of a row = codes of k = 2j (low nibble) and 2j + 1 (high nibble)
void launch_pack_nibbles(const uint8_t* src, uint8_t* dst, int K, int N, int n_off, cudaStream_t st, int il_group = 0,
                         int il_second = 0, int perm_dh = 0);
void launch_permute_scales(const float* src, float* dst, int N, int n_off, int perm_dh, cudaStream_t st);
// Y[r][n] = act( sum_d X[r][d] * W[(w_row_off + d)][n] + bias[n] + add[n] ), r < R
void launch_rows_gemm(const float* X, int ldx, const void* W, int w_kind, int w_row_off, int N, int K, const float* bias,
                      const float* add, int act_swish, float* Y, int ldy, int R, cudaStream_t st);
void launch_sinusoid(float* tau, int n_steps, int D, double min_period, double max_period, cudaStream_t st);
void launch_rope_table(float2* tab, int n_pos, int dh, double theta, cudaStream_t st);
// gains[d] = 1 + gamma[d]
void launch_one_plus(const float* gamma, float* out, int n, cudaStream_t st);
// mod rows [R][3D] (scale|shift|gate) -> in place (1+scale|shift|gate)
void launch_mod_finish(float* mod, int R, int D, cudaStream_t st);

// ---- per-call / per-step small kernels ---------------------------------------------------------
void launch_begin(const Request* rq, const int* status, const float* Ws, const float* bs, float* state_tok,
                  const Dims& d, int batch, cudaStream_t st);
// pi0: u[r][n] = swish(x[r] . Wc[:,n] + tb[n]) for the B*H action rows (+ state rows of h)
void launch_embed_pi0(const Request* rq, const int* status, const float* Wc, const float* tb, const float* state_tok,
                      float* h, float* u_f32, __nv_bfloat16* u_tiled, int rows_pad, const Dims& d, int batch,
                      cudaStream_t st);
// pi0.5: h[b*S+ns+i][n] = x . Wa[:,n] + ba[n] (+ state rows)
void launch_embed_pi05(const Request* rq, const int* status, const float* Wa, const float* ba, const float* state_tok,
                       float* h, const Dims& d, int batch, cudaStream_t st);
// n = h * rsqrt(mean h^2 + eps) * gain + shift  -> fp32 row-major or tiled bf16
// Pending split-K partial sums of the residual stream: n slabs of [M][D] floats, `stride` floats apart.  The kernel
// that reads h next adds them to each row in slab order (a fixed order: results are reproducible run to run) and,
// for the norms, writes the row back.
struct SlabSum {
  const float* slab;
  int n;
  size_t stride;
};
// (W8A8, widths for which rmsnorm_quantizes() holds: with out8 / xscale set the row leaves as its per-token e4m3
// quantization, codes in the tiled e4m3 layout, instead of as bf16)
bool rmsnorm_quantizes(int D);
void launch_rmsnorm(const int* status, float* h, const float* gain, const float* shift, float* out_f32,
                    __nv_bfloat16* out_tiled, int rows_pad, int M, int D, float eps, cudaStream_t st,
                    SlabSum slabs = SlabSum{nullptr, 0, 0}, uint8_t* out8 = nullptr, float* xscale = nullptr);
// final norm -> out-proj -> Euler update x += dt * (v + bout)
void launch_final(const Request* rq, const int* status, const float* h, const float* gain, const float* shift,
                  const float* Wout, const float* bout, float dt, const Dims& d, int batch, cudaStream_t st);
// h[row] += pending slabs (no-op when there are none)
void launch_add_slabs(const int* status, float* h, int M, int D, cudaStream_t st, SlabSum slabs);

// ---- CUDA-core GEMM (fp32 FMA) -----------------------------------------------------------------
enum : int { EPI_STORE = 0, EPI_SWISH = 1, EPI_RESID = 2, EPI_GEGLU = 3 };
struct SimtGemm {
  const float* A; int lda;        // [M][K] row-major
  const float* B; const float* B2;  // [K][N] row-major (B2: "up" matrix of GeGLU)
  int M, N, K;
  int epi;
  const float* bias;              // [N] or null (STORE / SWISH)
  const float* gate;              // [N] or null (RESID)
  float* out; int ldo;
  int rows_in, rows_out, row_off; // output row = (m / rows_in) * rows_out + row_off + m % rows_in
  int gelu_exact;
};
void launch_simt_gemm(const int* status, const SimtGemm& g, cudaStream_t st);

// ---- CUDA-core attention -----------------------------------------------------------------------
void launch_attention_simt(const Request* rq, const int* status, const float* qkv, const float2* rope, int layer,
                           int kv_is_bf16, float* out_f32, __nv_bfloat16* out_tiled, int rows_pad, const Dims& d,
                           int batch, cudaStream_t st);

// ---- tensor-core attention (mma.sync, bulk-copy staged K/V) ------------------------------------------
bool attention_mma_supported(const Dims& d);
int attention_pick_splits(const Dims& d, int batch, int max_prefix);
size_t attention_scratch_floats(const Dims& d, int batch, int splits);  // split-KV partials (O, m, l)
cudaError_t launch_attention_mma(const Request* rq, int* status, const float* qkv, const float2* rope, int layer,
                                 __nv_bfloat16* out_tiled, int rows_pad, int num_splits, float* scratch, const Dims& d,
                                 int batch, unsigned wait_limit, cudaStream_t st);

// ---- tcgen05 attention (large batches: two heads per CTA, whole key range, no split) ------------------
bool attention_tc_supported(const Dims& d);
// Output projection fused into the cluster attention kernel: packed weight blocks of the layer, optional per-channel
// weight scale and residual gate, and the slab array [Hq][rows][D] that receives one partial per head.
struct AttnOproj {
  const __nv_bfloat16* wo;
  const float* scale;
  const float* gate;
  float* slab;
  size_t slab_stride;
};
bool attention_oproj_supported(const Dims& d);
cudaError_t launch_attention_cluster(const Request* rq, int* status, const float* qkv, const float2* rope,
                                     const __nv_bfloat16* qr, const __nv_bfloat16* kr, const __nv_bfloat16* vr, int layer,
                                     __nv_bfloat16* out_tiled, int rows_pad, const Dims& d, int batch, unsigned wait_limit,
                                     cudaStream_t st, const AttnOproj* op = nullptr, unsigned long long* trace = nullptr);
// ---- tcgen05 attention for very few requests: key range split over a cluster of 8, two heads per CTA (attention_b1.cu)
bool attention_b1_supported(const Dims& d);
cudaError_t launch_attention_b1(const Request* rq, int* status, const __nv_bfloat16* q_tiles, const __nv_bfloat16* kr,
                                const __nv_bfloat16* vr, int layer, __nv_bfloat16* out_tiled, int rows_pad, const Dims& d,
                                int batch, int hpc, unsigned wait_limit, cudaStream_t st, unsigned long long* trace = nullptr,
                                int trace_all = 0);
// CTAs of one launch with `hpc` (1 or 2) query heads per CTA
int attention_b1_ctas(const Dims& d, int batch, int hpc);
cudaError_t launch_attention_tc(const Request* rq, int* status, const __nv_bfloat16* qr, const __nv_bfloat16* kr,
                                const __nv_bfloat16* vr, int layer, __nv_bfloat16* out_tiled, int rows_pad, const Dims& d,
                                int batch, const int* order, unsigned wait_limit, cudaStream_t st, unsigned long long* trace = nullptr,
                                int num_splits = 1, float* scratch = nullptr);
// key-range splits for grids far below one wave (1 = none)
int attention_tc_splits(const Dims& d, int batch, int n_sm, int max_prefix);
// combines split-KV partials ([b][head][split][64][dh] unnormalised rows, then [..][64][2] (max in log2 units, sum))
cudaError_t launch_attention_merge(int* status, const float* part_o, const float* part_ml, __nv_bfloat16* out, int rows_pad,
                                   int num_splits, const Dims& d, int batch, cudaStream_t st);

// ---- tcgen05 GEMM ------------------------------------------------------------------------------
enum : int { TC_STORE = 0, TC_RESID = 1, TC_GEGLU = 2, TC_BIAS_ROWMAP = 3, TC_QKV_ROT = 4, TC_GEGLU_IL = 5 };
struct TcGemm {
  const __nv_bfloat16* W;   // packed blocks [N/128][KC][128x64]
  const __nv_bfloat16* W2;  // second matrix (GeGLU "up"), same packing, or null
  const __nv_bfloat16* X;   // tiled activations [KC][rows_pad][64]
  int rows_pad, M, N, K;
  int epi;
  const float* scale;  // per-out-channel dequant scale or null
  // W8A8: W and X hold e4m3 codes (128-byte rows = 128 k per block / tile chunk), the product runs on the FP8 tensor
  // path and every accumulator column is multiplied by its token's activation scale
  int fp8;
  unsigned long long* trace;   // or null: every CTA stamps into slot (linear block index) x 16: start, set-up done,
                               // dependency resolved, first operands landed, MMAs issued, accumulator complete, stores
                               // done, (SM id)
  const float* xscale;   // [rows] per-token activation scale (fp8 only)
  const float* scale2;
  const float* bias;   // TC_BIAS_ROWMAP
  const float* gate;   // TC_RESID (null = 1)
  float* out_f32; int ldo;          // TC_STORE / TC_RESID / TC_BIAS_ROWMAP
  __nv_bfloat16* out_tiled;         // TC_GEGLU: [N/64][rows_pad][64]; TC_GEGLU_IL: W holds gate and up interleaved in groups
                                    // of 64 channels (N = 2 x mlp_dim packed rows), one 64-channel k-chunk of output per tile
  int rows_in, rows_out, row_off;   // TC_BIAS_ROWMAP row remap
  int gelu_exact;
  int splits;                       // split-K factor (TC_RESID only)
  float* slab;                      // TC_RESID with splits > 1: when set, k-range z stores its partial tile to
                                    // slab[z][M][ldo] (summed by the next reader of h) instead of reducing into out_f32
  int nt_override;                  // host side: token-tile width chosen for this GEMM (0 = the caller's default)
  int perm_dh, perm_end;            // TC_STORE: packed rows < perm_end map to channels by qkv_packed_to_channel
  // TC_QKV_ROT: the fused q|k|v projection (rows packed by qkv_channel_to_packed) leaves the kernel as the
  // attention kernel's operands: q rotated and scaled by 1/sqrt(dh), k rotated, v as is, all bf16,
  // q [b][Hq][S][dh], k and v [b][Hkv][S][dh]; token t is suffix row t % S of request t / S at position
  // prefix_len(request) + t % S.
  const Request* rq;
  const float2* rope;               // [pos][dh/2] (cos, sin) or null (no rotation)
  __nv_bfloat16 *qr, *kr, *vr;
  int S, Hq, Hkv, dh;
  unsigned wait_limit;
};
// Returns cudaSuccess or the launch error; `nt` is the token-tile width (64, 128 or 256).
cudaError_t launch_tc_gemm(int* status, const TcGemm& g, int nt, cudaStream_t st);
cudaError_t tc_gemm_setup();  // one-time attribute setup (dynamic shared memory opt-in)

// Persistent tile GEMM (gemm_persist.cu): 128-row weight tiles x 256-token tiles, two accumulators in tensor memory so
// that the epilogue of a tile overlaps the main loop of the next.  The rows of every weight tile are interleaved in
// groups of 16: rows 32 q + i (i < 16) and 32 q + 16 + i are combined by the epilogue.
//   gate / up (qkv = 0): the tile holds 64 channels, gate rows at 32 q + i and up rows at 32 q + 16 + i of channel
//     16 q + i; N = 2 x mlp_dim; out_tiled gets gelu(gate) * up.
//   q | k | v (qkv = 1): the packing of qkv_channel_to_packed (64 first-half channels of a head, then their rotary
//     partners; v: 128 channels) with packed row r of a tile moved to row 32 ((r % 64) / 16) + 16 (r / 64) + r % 16;
//     q rotated and scaled by 1 / sqrt(dh), k rotated, v as is, all bf16, laid out as for TC_QKV_ROT.
struct PersistGemm {
  const __nv_bfloat16* W;       // (N / 128) tiles x KC blocks of 128 rows x 128 bytes (bf16 or e4m3)
  const __nv_bfloat16* X;       // tiled activations [KC][rows_pad][128 bytes]
  __nv_bfloat16* out_tiled;     // gate / up: [N / 128][rows_pad][64] bf16, 16-byte chunks swizzled by row & 7
  const float* scale_g;         // per-channel weight scales or null (q | k | v: per packed row, un-interleaved order)
  const float* scale_u;
  const float* xscale;          // fp8: per-token activation scales
  int M, N, K, rows_pad;
  int gelu_exact, fp8, qkv;
  unsigned wait_limit;
  unsigned long long* trace;    // or null: CTA b stamps slot b (16 words)
  const Request* rq;            // q | k | v
  const float2* rope;
  __nv_bfloat16 *qr, *kr, *vr;
  int S, Hq, Hkv, dh;
};
bool persist_gemm_supported(int M, int N, int K, int rows_pad, bool fp8);
int persist_gemm_ctas(const PersistGemm& g, int n_sm);
cudaError_t persist_gemm_setup();
cudaError_t launch_persist_gemm(int* status, const PersistGemm& g, int n_sm, cudaStream_t st);
// ---- cluster split-K GEMM for a single 64-token tile (gemm_b1.cu) --------------------------------------------
enum : int { B1_QKV = 0, B1_GEGLU = 1, B1_RESID = 2 };
struct B1Gemm {
  const __nv_bfloat16* W;    // packed blocks [N/128][K/64][128x64]
  int w_bits;                // 8 (e4m3 codes) or 4 (int4 codes: blocks of [128 rows][32 bytes], byte j of a row = codes of
                             // k = 2j (low nibble) and 2j + 1) when W8 is set
  const uint8_t* W8;         // or: e4m3 codes, blocks [N/128][K/64][128 rows][64 bytes] in the same row order, decoded
                             // to bf16 inside the kernel (one byte per weight crosses HBM); scales as below
  const __nv_bfloat16* X;    // tiled activations [K/64][64][64] (64-row tiles, back to back)
  int N, K, M;               // packed rows, contraction length, valid tokens (<= 64)
  int epi;
  int nk_max;                // (set by the launcher) most k-steps of one CTA
  const float* wscale;       // per packed row dequant scale or null (B1_GEGLU: per gate channel f)
  const float* wscale2;      // B1_GEGLU: per up channel f
  // norm folded into this projection: X holds bf16(h * gain); the accumulator columns are multiplied by
  // rsqrt(sum_i ss_part[i][token] * inv_D + eps) and shift_row (per packed row: shift . W) is added.  ss_part == null:
  // X is already normalised.
  const float* ss_part;
  int ss_n;
  float inv_D, eps;
  const float* shift_row;
  // B1_QKV: see TcGemm (TC_QKV_ROT)
  const Request* rq;
  const float2* rope;
  __nv_bfloat16 *qr, *kr, *vr;
  __nv_bfloat16* q_tiles;    // set: q goes out as the cluster attention kernel's operand tiles instead of rows (qr)
  int S, Hq, Hkv, dh;
  int Sk_stride, koff;       // key rows per (request, kv head) in kr / vr and the key row of query row 0 (see Dims)
  // B1_GEGLU: W holds gate and up interleaved in groups of 64 channels; output [N/128][64][64] tiled
  __nv_bfloat16* out_tiled;
  int gelu_exact;
  // B1_RESID: h[token][n] += gate[n] * scale[n] * acc; then, when xn_out is set, the operands of the norm that
  // follows: xn_out = bf16(h * gain_next) in the tiled layout and ss_out[N/128][64] partial sums of squares
  float* h;
  int ldh;
  const float* gate;
  const float* gain_next;
  __nv_bfloat16* xn_out;
  float* ss_out;
  // B1_RESID as the second layer of the pi0 action / time MLP: with `bias` set, h is written, not updated --
  // h[token][n] = bias[n] + scale[n] * acc for action rows, h = state_tok[request][n] for the first `ns` rows of every
  // request's S suffix rows (the state tokens, whose embedding does not pass through the MLP)
  const float* bias;
  const float* state_tok;
  int ns;
  unsigned wait_limit;
  int trace_all;               // every CTA stamps, into slot (linear CTA index) of `trace`
  unsigned long long* trace;   // 16-entry slot of this launch or null: start, set-up done, dependency resolved, MMAs
                               // complete, partials received, epilogue done, cluster released, (SM id)
};
// ---- step boundary of the single-tile loop (step_b1.cu): velocity head + Euler update of step k - 1, suffix embedding
// of step k, one cluster of D / 128 CTAs -----------------------------------------------------------------------------
struct StepB1 {
  const Request* rq;
  int batch, S, H, ns, A, D, M;   // M = batch * S token rows (<= 64)
  float eps;
  int first, last;                // first: no head (the actions are the noise); last: no embedding
  const float* h_in;              // [M][D] residual stream after the last layer
  const float* gain_f;            // final norm: gain (1 + gamma or 1 + scale) and shift or null
  const float* shift_f;
  const float* Wout;              // [D][A]
  const float* bout;              // [A]
  float dt;
  int ada;                        // 0: pi0 (u = swish(x Wc + bias) -> bf16 tile), 1: pi0.5 (h = x Wc + bias, + norm operands)
  const float* Wc;                // [A][D]
  const float* bias;              // [D]
  const float* state_tok;         // [batch][D]
  __nv_bfloat16* u;               // pi0: tiled [D/64][64][64], row = token row
  float* h_out;                   // pi0.5: [M][D]
  const float* gain_next;         // pi0.5: gain of the first norm of layer 0
  __nv_bfloat16* xn_out;          // pi0.5: bf16(h * gain_next), tiled
  float* ss_out;                  // pi0.5: [D/128][64] partial sums of squares
  unsigned wait_limit;
  unsigned long long* trace;      // 16-entry slot or null: start, constants fetched, dependency resolved, slice
                                  // staged, partial formed, partials received, embedding stored
};
bool step_b1_supported(const Dims& d, int batch);
cudaError_t launch_step_b1(int* status, const StepB1& p, cudaStream_t st);
int b1_pick_cluster(int tiles, int KC, int n_sm);
bool b1_gemm_supported(int N, int K, int C, int n_sm, bool qkv);
cudaError_t launch_b1_gemm(int* status, const B1Gemm& g, int C, cudaStream_t st);
// out[n] = scale(n) * sum_k shift[k] * W[n][k] for the packed rows n < N of a packed matrix with K / 64 chunks.
// interleaved = 1: the rows are gate / up channels interleaved in groups of 64 (scale per gate channel f = wscale[f],
// per up channel wscale2[f]); otherwise scale(n) = wscale[n].  Null scales mean 1.
void launch_shift_rows(const float* shift, const __nv_bfloat16* Wp, const float* wscale, const float* wscale2,
                       int interleaved, float* out, int N, int K, cudaStream_t st);

}  // namespace phyai
