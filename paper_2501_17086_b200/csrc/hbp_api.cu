// C ABI of libhbp: configuration checks, workspace carve-up and the kernel sequences of
// hbp_forward / hbp_backward / hbp_exact.  No device memory is allocated here; every buffer is either
// the caller's or a slice of the caller's workspace.
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "hbp_internal.h"

namespace hbp {
bool gemm(Launcher& lc, const GemmArgs& g, int* status_word) {
  if (!lc.force_simt && !g.relu && gemm_tc(lc, g, status_word)) return true;
  gemm_simt(lc, g);
  return false;
}
}  // namespace hbp

using namespace hbp;

struct ProfSeg {
  cudaEvent_t beg, end;
  int phase;
  int64_t launches;
};

struct hbp_ctx {
  hbp_config cfg;
  // kernel-selection modes, read from the environment (HBP_FORCE_SIMT=1, HBP_GEMM_PAIR=0, HBP_SCAN_OPERAND=0) when
  // THIS context is created and kept with it: another context created later under other settings does not change them
  bool force_simt = false, gemm_pair = false, scan_operand = true;
  bool profiling = false;
  std::vector<ProfSeg> segs;       // recorded, not yet read
  std::vector<ProfSeg> free_segs;  // event pairs ready for reuse
  char* ws = nullptr;
  size_t ws_bytes = 0;
  bool forward_done = false;
  int64_t launches = 0;
  int es = 4;         // element size
  int steps = 0;      // residual steps seen by the scan
  int layers = 0;     // MLP layers (== steps for MLP kinds, decoder blocks for the Transformer)
  int group = 1;      // layers whose hidden-size scratch is materialised at once
  bool preln = false;
  // workspace slices (nullptr when unused)
  int* status = nullptr;
  char* Y = nullptr;       // [steps][N][d] LayerNorm output xhat
  float* rstd = nullptr;   // [steps][N]
  char* ACT = nullptr;     // [layers][N][h] gelu(Z)
  char* DACT = nullptr;    // [layers][N][h] gelu'(Z)
  float* xres = nullptr;   // [N][d] float master of the residual stream (bf16 only)
  double* hres = nullptr;  // RNN: 2 x [B][d] double master of the recurrent state (ping-pong)
  double* Pd = nullptr;    // tanh RNN: [T][B][d] input projections U x_t in double for the one-launch recurrence
  // RNN, float: tf32 high/low splits of the GEMM operands, each written with the contraction index
  // contiguous: A* is g * tanh' as [T*B][d] for the VJP or [d][T*B] for the weight gradients, H* the states
  // h_0..h_{T-1} as [d][T*B], X* the inputs as [in][T*B], W* the recurrent matrix transposed
  float *Ahi = nullptr, *Alo = nullptr, *Hhi = nullptr, *Hlo = nullptr, *Xhi = nullptr, *Xlo = nullptr;
  float *Whi = nullptr, *Wlo = nullptr;
  char* U = nullptr;       // [steps][N][d] block VJP outputs (dY before the LayerNorm finish)
  char* H1 = nullptr;      // [group][N][h] dZ
  float2* lnpart = nullptr;  // [steps][N][slots] partial row sums of dY and dY * xhat from the GEMM epilogue
  float4* lnstat = nullptr;  // [steps][N] {rstd, mean dY, mean dY * xhat, 0}
  int ln_slots = 0;
  char* C = nullptr;       // RNN: [T][B][d] tanh'(z_t) = 1 - tanh(z_t)^2
  // GRU: the update gate z_t [T][B][d] (the diagonal of K), the VJP coefficients [T*B][4d] = [c_r|c_z|c_nr|c_n]
  // and, for the GEMMs that do not take the tf32 splits, g times those coefficients [T*B][4d]
  char *Zc = nullptr, *C4 = nullptr, *A4 = nullptr;
  // LSTM (u = d / 2 units): the scan's gate [T][B][2u] = [f | 0], the VJP coefficients [T*B][5u] (A4 is [T*B][4u])
  char *Fg = nullptr, *C5 = nullptr;
  // ReLU(x + Block(x)): the masks [L][N][d] (0/1 in dtype: the scan's gate) and mask * g_{l+1} [L][N][d]
  char *MASK = nullptr, *GM = nullptr;
  // post-LN layers: GM holds LayerNorm-backward of g_{l+1} (what the block is differentiated against), CB the part of
  // the layer's VJP that is not the block's, rstd [L][N] is the scan's row gate
  char* CB = nullptr;
  char* scan_scratch = nullptr;
  size_t scan_scratch_bytes = 0;
  float* partial = nullptr;  // split-K / gate-gradient partial sums
  size_t partial_floats = 0;
  char* QKV = nullptr;     // [Lb][N][3d]
  char* O = nullptr;       // [Lb][N][d]
  float* lse = nullptr;    // [Lb][B][H][S]
  char* Wqkv = nullptr;    // [Lb][3d][d]
  char* dO = nullptr;      // [Lb][N][d]
  char* dQKV = nullptr;    // [Lb][N][3d]
  float* drow = nullptr;   // [Lb][B][H][S]
  float2* dopart = nullptr;  // [Lb][N][do_slots] row sums of dO and dO * O per 64 columns (= per head)
  int do_slots = 0;
};

namespace {

constexpr size_t kAlign = 256;
constexpr int kGateBlocks = 256;
constexpr int kMaxSplit = 256;

inline size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

hbp_status check_config(const hbp_config* c) {
  if (!c) return HBP_ERR_INVALID_ARG;
  if (c->dtype != HBP_F32 && c->dtype != HBP_BF16) return HBP_ERR_DTYPE;
  if (c->block < 0 || c->block > HBP_BLOCK_POSTLN_MLP) return HBP_ERR_UNSUPPORTED;
  if (c->gate < 0 || c->gate > HBP_GATE_CHANNEL_PER_STEP) return HBP_ERR_UNSUPPORTED;
  if (c->loss != HBP_LOSS_FINAL && c->loss != HBP_LOSS_EVERY_STEP) return HBP_ERR_UNSUPPORTED;
  const int v = c->dtype == HBP_F32 ? 4 : 8;
  if (c->L <= 0 || c->d <= 0 || c->tokens <= 0) return HBP_ERR_SHAPE;
  if (!(c->gamma >= 0.0f && c->gamma <= 1.0f)) return HBP_ERR_INVALID_ARG;
  if (c->gamma != 0.0f && (c->gate != HBP_GATE_ONE || c->block == HBP_BLOCK_RNN_TANH)) return HBP_ERR_UNSUPPORTED;
  if (c->d % v) return HBP_ERR_SHAPE;
  if (c->d / v > 1024) return HBP_ERR_SHAPE;  // one block per row in the LayerNorm kernels
  const bool gated_cell = c->block == HBP_BLOCK_GRU || c->block == HBP_BLOCK_LSTM;
  if ((gated_cell || c->block == HBP_BLOCK_RELU_MLP) && (c->gate != HBP_GATE_ONE || c->gamma != 0.0f)) return HBP_ERR_UNSUPPORTED;
  if (c->block == HBP_BLOCK_POSTLN_MLP && c->gate != HBP_GATE_ONE) return HBP_ERR_UNSUPPORTED;
  // the 0/1 mask is a sign decision: taken in bf16 arithmetic it differs from an exact evaluation on the elements
  // that land near zero, and each such element changes its whole gradient path; float only
  if (c->block == HBP_BLOCK_RELU_MLP && c->dtype != HBP_F32) return HBP_ERR_UNSUPPORTED;
  if (c->block == HBP_BLOCK_LSTM && (c->hidden <= 0 || c->hidden % v || 2 * c->hidden != c->d)) return HBP_ERR_SHAPE;
  if (c->block == HBP_BLOCK_RNN_TANH || gated_cell) {
    if (c->in_dim <= 0 || c->in_dim % v) return HBP_ERR_SHAPE;
    if (c->batch != c->tokens) return HBP_ERR_SHAPE;
  } else {
    if (c->hidden <= 0 || c->hidden % v) return HBP_ERR_SHAPE;
  }
  if (c->block == HBP_BLOCK_PRELN_TRANSFORMER) {
    if (c->n_heads <= 0 || c->head_dim <= 0 || c->seq <= 0 || c->batch <= 0) return HBP_ERR_SHAPE;
    if ((int64_t)c->n_heads * c->head_dim != c->d) return HBP_ERR_SHAPE;
    if ((int64_t)c->batch * c->seq != c->tokens) return HBP_ERR_SHAPE;
    if (c->head_dim != 32 && c->head_dim != 64 && c->head_dim != 128) return HBP_ERR_UNSUPPORTED;
  }
  return HBP_OK;
}

// Lays the workspace out; with base == nullptr only the total size is computed.
size_t carve(hbp_ctx* c, char* base) {
  const hbp_config& f = c->cfg;
  size_t off = 0;
  auto take = [&](size_t bytes) -> char* {
    char* p = base ? base + off : nullptr;
    off += align_up(bytes);
    return p;
  };
  const size_t es = f.dtype == HBP_F32 ? 4 : 2;
  const size_t N = (size_t)f.tokens, d = (size_t)f.d, h = (size_t)f.hidden;
  c->es = (int)es;
  c->preln = f.block == HBP_BLOCK_PRELN_MLP || f.block == HBP_BLOCK_PRELN_TRANSFORMER;
  c->steps = f.block == HBP_BLOCK_PRELN_TRANSFORMER ? 2 * f.L : f.L;
  c->layers = f.L;
  const size_t steps = (size_t)c->steps;
  c->status = (int*)take(256);
  c->U = take(steps * N * d * es);
  const bool recurrent = f.block == HBP_BLOCK_RNN_TANH || f.block == HBP_BLOCK_GRU || f.block == HBP_BLOCK_LSTM;
  if (f.dtype == HBP_BF16 && !recurrent) c->xres = (float*)take(N * d * 4);
  c->partial_floats = (size_t)kGateBlocks * d;
  if (f.block == HBP_BLOCK_LSTM) {
    const size_t in = (size_t)f.in_dim, u = d / 2, rows = steps * N;
    c->Fg = take(rows * d * es);
    c->C5 = take(rows * 5 * u * es);
    c->A4 = take(rows * 4 * u * es);
    c->hres = (double*)take(2 * N * d * 8);
    if (f.dtype == HBP_F32) {
      c->Ahi = (float*)take(rows * 4 * u * 4); c->Alo = (float*)take(rows * 4 * u * 4);
      c->Hhi = (float*)take(rows * u * 4); c->Hlo = (float*)take(rows * u * 4);
      c->Xhi = (float*)take(rows * in * 4); c->Xlo = (float*)take(rows * in * 4);
      c->Whi = (float*)take(4 * u * u * 4); c->Wlo = (float*)take(4 * u * u * 4);
    }
    c->scan_scratch_bytes = scan_scratch_bytes(f.dtype, f.L, f.tokens, f.d);
    c->scan_scratch = take(c->scan_scratch_bytes);
    const size_t wmax = 4 * u * (u > in ? u : in);
    if ((size_t)kMaxSplit * wmax > c->partial_floats) c->partial_floats = (size_t)kMaxSplit * wmax;
  } else if (f.block == HBP_BLOCK_GRU) {
    const size_t in = (size_t)f.in_dim;
    c->Zc = take(steps * N * d * es);
    c->C4 = take(steps * N * 4 * d * es);
    c->A4 = take(steps * N * 4 * d * es);
    c->hres = (double*)take(2 * N * d * 8);
    if (f.dtype == HBP_F32) {
      c->Ahi = (float*)take(steps * N * 4 * d * 4); c->Alo = (float*)take(steps * N * 4 * d * 4);
      c->Hhi = (float*)take(steps * N * d * 4); c->Hlo = (float*)take(steps * N * d * 4);
      c->Xhi = (float*)take(steps * N * in * 4); c->Xlo = (float*)take(steps * N * in * 4);
      c->Whi = (float*)take(3 * d * d * 4); c->Wlo = (float*)take(3 * d * d * 4);
    }
    c->scan_scratch_bytes = scan_scratch_bytes(f.dtype, f.L, f.tokens, f.d);
    c->scan_scratch = take(c->scan_scratch_bytes);
    const size_t wmax = 3 * d * (d > in ? d : in);
    if ((size_t)kMaxSplit * wmax > c->partial_floats) c->partial_floats = (size_t)kMaxSplit * wmax;
  } else if (f.block == HBP_BLOCK_RNN_TANH) {
    c->C = take(steps * N * d * es);
    c->hres = (double*)take(2 * N * d * 8);
    if (f.gate != HBP_GATE_CHANNEL_PER_STEP) {
      const size_t pb = rnn_persistent_proj_bytes(f.L, f.tokens, f.d);
      if (pb) c->Pd = (double*)take(pb);
    }
    if (f.dtype == HBP_F32) {
      c->Ahi = (float*)take(steps * N * d * 4); c->Alo = (float*)take(steps * N * d * 4);
      c->Hhi = (float*)take(steps * N * d * 4); c->Hlo = (float*)take(steps * N * d * 4);
      c->Xhi = (float*)take(steps * N * (size_t)f.in_dim * 4); c->Xlo = (float*)take(steps * N * (size_t)f.in_dim * 4);
      c->Whi = (float*)take(d * d * 4); c->Wlo = (float*)take(d * d * 4);
    }
    c->scan_scratch_bytes = scan_scratch_bytes(f.dtype, f.L, f.tokens, f.d);
    c->scan_scratch = take(c->scan_scratch_bytes);
    const size_t wmax = d * (d > (size_t)f.in_dim ? d : (size_t)f.in_dim);
    if ((size_t)kMaxSplit * wmax > c->partial_floats) c->partial_floats = (size_t)kMaxSplit * wmax;
  } else {
    if (c->preln) {
      c->Y = take(steps * N * d * es);
      c->rstd = (float*)take(steps * N * 4);
      if (f.dtype == HBP_BF16) {
        c->ln_slots = gemm_tc_stats_slots(f.d);
        c->lnpart = (float2*)take(steps * N * c->ln_slots * sizeof(float2));
        c->lnstat = (float4*)take(steps * N * sizeof(float4));
      }
    }
    if (f.block == HBP_BLOCK_RELU_MLP) {
      c->MASK = take(steps * N * d * es);
      c->GM = take(steps * N * d * es);
    }
    if (f.block == HBP_BLOCK_POSTLN_MLP) {
      c->GM = take(steps * N * d * es);
      c->CB = take(steps * N * d * es);
      c->rstd = (float*)take(steps * N * 4);
    }
    c->ACT = take((size_t)c->layers * N * h * es);
    c->DACT = take((size_t)c->layers * N * h * es);
    const size_t per_layer = N * h * es;
    size_t grp = ((size_t)6 << 30) / per_layer;
    if (grp < 1) grp = 1;
    if (grp > (size_t)c->layers) grp = (size_t)c->layers;
    c->group = (int)grp;
    c->H1 = take(grp * per_layer);
  }
  if (f.block == HBP_BLOCK_PRELN_TRANSFORMER) {
    const size_t Lb = (size_t)f.L;
    c->QKV = take(Lb * N * 3 * d * es);
    c->O = take(Lb * N * d * es);
    c->lse = (float*)take(Lb * (size_t)f.batch * f.n_heads * f.seq * 4);
    c->Wqkv = take(Lb * 3 * d * d * es);
    c->dO = take(Lb * N * d * es);
    c->dQKV = take(Lb * N * 3 * d * es);
    c->drow = (float*)take(Lb * (size_t)f.batch * f.n_heads * f.seq * 4);
    if (f.dtype == HBP_BF16 && f.head_dim == 64) {
      c->do_slots = gemm_tc_stats_slots(f.d);
      c->dopart = (float2*)take(Lb * N * c->do_slots * sizeof(float2));
    }
  }
  c->partial = (float*)take(c->partial_floats * 4);
  return off;
}

struct Run {
  hbp_ctx* c;
  Launcher lc;
  const hbp_params* p;
  const char* x_all;
  const char* inputs;
  char* g;
  const char* delta;
  int64_t N, d, h, es, state;  // state = N*d elements
  Run(hbp_ctx* ctx, const hbp_params* params, void* stream) : c(ctx), p(params) {
    lc.stream = (cudaStream_t)stream;
    lc.launches = &ctx->launches;
    lc.force_simt = ctx->force_simt;
    lc.gemm_pair = ctx->gemm_pair;
    N = ctx->cfg.tokens;
    d = ctx->cfg.d;
    h = ctx->cfg.hidden;
    es = ctx->es;
    state = N * d;
    x_all = inputs = delta = nullptr;
    g = nullptr;
  }
  const char* at(const void* base, int64_t elems) const { return (const char*)base + elems * es; }
  char* at(void* base, int64_t elems) const { return (char*)base + elems * es; }
  const void* gate_ptr(int step) const {
    if (c->cfg.gate == HBP_GATE_ONE) return nullptr;
    return at(p->a, c->cfg.gate == HBP_GATE_CHANNEL_PER_STEP ? (int64_t)step * d : 0);
  }
  GemmArgs base_args() const {
    GemmArgs a;
    a.in_dtype = c->cfg.dtype;
    return a;
  }
  bool u_has_delta = false;  // the VJP GEMM already added delta_l to u_l
  // float tanh RNN: the scan before an all-step VJP may write that VJP's split operand as a by-product
  bool want_operand = false;       // set by the iteration loop: another all-step VJP follows the next scan
  mutable bool operand_ready = false;  // set by the scan when it did
  int rnn_tc = -1;                     // see rnn_operand_from_scan
  bool shifted = false;      // Highway-BP call on a config with gamma > 0 (exact BP ignores the shift)
  bool stats_ok = true;  // every dY GEMM since the last reset also produced the LayerNorm row sums
  bool run_gemm(const GemmArgs& a) { return gemm(lc, a, c->status); }
  hbp_status result() const { return lc.err == cudaSuccess ? HBP_OK : HBP_ERR_CUDA; }

  // state/step index of MLP layer b and of attention layer b
  int mlp_step(int b) const { return c->cfg.block == HBP_BLOCK_PRELN_TRANSFORMER ? 2 * b + 1 : b; }
  int step_stride() const { return c->cfg.block == HBP_BLOCK_PRELN_TRANSFORMER ? 2 : 1; }
  // operand of W1 for layer b: LayerNorm output or the raw state
  const char* mlp_operand(int b) const {
    return c->preln ? at(c->Y, (int64_t)mlp_step(b) * state) : at(x_all, (int64_t)mlp_step(b) * state);
  }

  // Asks the dY GEMM (first step `step`, `ss` steps between batch entries) for the LayerNorm row sums too.
  void ln_epilogue(GemmArgs& b, int step, int ss) {
    if (!c->lnpart) return;
    b.epi = EPI_STORE_LN;
    b.E = at(c->Y, (int64_t)step * state); b.lde = d; b.e_sb = ss * state;
    b.stats = c->lnpart + (int64_t)step * N * c->ln_slots;
    b.stats_sb = (int64_t)ss * N * c->ln_slots;
  }

  // What the MLP block of layer b0 is differentiated against: g_{l+1}, or mask_l * g_{l+1} for ReLU(x + Block(x))
  // (mask_gradients fills GM first).
  const char* upstream(int b0) const {
    if (c->GM) return at(c->GM, (int64_t)b0 * state);
    return at(g, (int64_t)(mlp_step(b0) + 1) * state);
  }
  void mask_gradients(int b0, int b1) {
    if (!c->GM) return;
    if (c->CB) {  // post-LN: through the layer's LayerNorm first (its output is the next state)
      postln_prepass(lc, c->cfg.dtype, at(g, (int64_t)(b0 + 1) * state), at(x_all, (int64_t)(b0 + 1) * state),
                     c->rstd + (int64_t)b0 * N, at(c->GM, (int64_t)b0 * state), at(c->CB, (int64_t)b0 * state),
                     (int64_t)(b1 - b0) * N, (int)d);
      return;
    }
    mul_elementwise(lc, c->cfg.dtype, at(c->GM, (int64_t)b0 * state), at(c->MASK, (int64_t)b0 * state),
                    at(g, (int64_t)(b0 + 1) * state), (int64_t)(b1 - b0) * state);
  }

  // ---- MLP block: u = J^T g for layers [b0, b1) (b1 - b0 <= group), from states g[step+1] -------
  // dA = G W2, dZ = dA * gelu'(Z) -> H1 (cached derivative);  dY = dZ W1 -> U[step].
  void mlp_vjp(int b0, int b1, bool want_dy) {
    const int nb = b1 - b0, ss = step_stride();
    GemmArgs a = base_args();
    a.M = (int)N; a.N = (int)h; a.K = (int)d; a.batch = nb;
    a.A = upstream(b0); a.a_sm = d; a.a_sk = 1; a.a_sb = ss * state;
    a.B = at(p->W2, (int64_t)b0 * d * h); a.b_sn = 1; a.b_sk = h; a.b_sb = d * h;
    a.epi = EPI_MUL;
    a.E = at(c->DACT, (int64_t)b0 * N * h); a.lde = h; a.e_sb = N * h;
    a.D = c->H1; a.ldd = h; a.d_sb = N * h;
    run_gemm(a);
    if (!want_dy) return;
    GemmArgs b = base_args();
    b.M = (int)N; b.N = (int)d; b.K = (int)h; b.batch = nb;
    b.A = c->H1; b.a_sm = h; b.a_sk = 1; b.a_sb = N * h;
    b.B = at(p->W1, (int64_t)b0 * h * d); b.b_sn = 1; b.b_sk = d; b.b_sb = h * d;
    b.epi = EPI_STORE;
    b.D = at(c->U, (int64_t)mlp_step(b0) * state); b.ldd = d; b.d_sb = ss * state;
    ln_epilogue(b, mlp_step(b0), ss);
    const bool tc = run_gemm(b);
    stats_ok = stats_ok && (tc || !c->lnpart);
  }
  // dW2 = G^T gelu(Z), dW1 = dZ^T y for layers [b0, b1); needs dZ in H1 from mlp_vjp.
  void mlp_wgrad(int b0, int b1, const hbp_grads* gr) {
    const int nb = b1 - b0, ss = step_stride();
    GemmArgs a = base_args();
    a.M = (int)d; a.N = (int)h; a.K = (int)N; a.batch = nb;
    a.A = upstream(b0); a.a_sm = 1; a.a_sk = d; a.a_sb = ss * state;
    a.B = at(c->ACT, (int64_t)b0 * N * h); a.b_sn = 1; a.b_sk = h; a.b_sb = N * h;
    a.epi = EPI_STORE; a.d_f32 = true;
    a.D = gr->dW2 + (int64_t)b0 * d * h; a.ldd = h; a.d_sb = d * h;
    run_gemm(a);
    GemmArgs b = base_args();
    b.M = (int)h; b.N = (int)d; b.K = (int)N; b.batch = nb;
    b.A = c->H1; b.a_sm = 1; b.a_sk = h; b.a_sb = N * h;
    b.B = mlp_operand(b0); b.b_sn = 1; b.b_sk = d; b.b_sb = ss * state;
    b.epi = EPI_STORE; b.d_f32 = true;
    b.D = gr->dW1 + (int64_t)b0 * h * d; b.ldd = d; b.d_sb = h * d;
    run_gemm(b);
  }

  // ---- attention block of decoder layers [b0, b1) ------------------------------------------------
  void attn_vjp(int b0, int b1, bool want_dy) {
    const hbp_config& f = c->cfg;
    const int nb = b1 - b0;
    GemmArgs a = base_args();  // dO = G Wo
    a.M = (int)N; a.N = (int)d; a.K = (int)d; a.batch = nb;
    a.A = at(g, (int64_t)(2 * b0 + 1) * state); a.a_sm = d; a.a_sk = 1; a.a_sb = 2 * state;
    a.B = at(p->Wo, (int64_t)b0 * d * d); a.b_sn = 1; a.b_sk = d; a.b_sb = d * d;
    a.epi = EPI_STORE;
    a.D = at(c->dO, (int64_t)b0 * state); a.ldd = d; a.d_sb = state;
    if (c->dopart) {  // also the per-head row sums of dO * O that the attention backward needs
      a.epi = EPI_STORE_LN;
      a.E = at(c->O, (int64_t)b0 * state); a.lde = d; a.e_sb = state;
      a.stats = c->dopart + (int64_t)b0 * N * c->do_slots; a.stats_sb = N * c->do_slots;
    }
    const bool do_tc = run_gemm(a);
    AttnArgs t;
    t.dtype = f.dtype; t.batch = nb * f.batch; t.seq = f.seq; t.heads = f.n_heads; t.head_dim = f.head_dim;
    t.qkv = at(c->QKV, (int64_t)b0 * 3 * state);
    t.o = at(c->O, (int64_t)b0 * state);
    t.lse = c->lse + (int64_t)b0 * f.batch * f.n_heads * f.seq;
    t.d_o = at(c->dO, (int64_t)b0 * state);
    t.d_qkv = at(c->dQKV, (int64_t)b0 * 3 * state);
    t.delta_rows = c->drow + (int64_t)b0 * f.batch * f.n_heads * f.seq;
    t.status = c->status;
    if (c->dopart && do_tc) { t.d_stats = c->dopart + (int64_t)b0 * N * c->do_slots; t.d_slots = c->do_slots; }
    attention_bwd(lc, t);
    if (!want_dy) return;
    GemmArgs b = base_args();  // dY = [dQ dK dV] [Wq; Wk; Wv]
    b.M = (int)N; b.N = (int)d; b.K = (int)(3 * d); b.batch = nb;
    b.A = at(c->dQKV, (int64_t)b0 * 3 * state); b.a_sm = 3 * d; b.a_sk = 1; b.a_sb = 3 * state;
    b.B = at(c->Wqkv, (int64_t)b0 * 3 * d * d); b.b_sn = 1; b.b_sk = d; b.b_sb = 3 * d * d;
    b.epi = EPI_STORE;
    b.D = at(c->U, (int64_t)(2 * b0) * state); b.ldd = d; b.d_sb = 2 * state;
    ln_epilogue(b, 2 * b0, 2);
    const bool tc = run_gemm(b);
    stats_ok = stats_ok && (tc || !c->lnpart);
  }
  void attn_wgrad(int b0, int b1, const hbp_grads* gr) {
    const int nb = b1 - b0;
    GemmArgs a = base_args();  // dWo = G^T O
    a.M = (int)d; a.N = (int)d; a.K = (int)N; a.batch = nb;
    a.A = at(g, (int64_t)(2 * b0 + 1) * state); a.a_sm = 1; a.a_sk = d; a.a_sb = 2 * state;
    a.B = at(c->O, (int64_t)b0 * state); a.b_sn = 1; a.b_sk = d; a.b_sb = state;
    a.epi = EPI_STORE; a.d_f32 = true;
    a.D = gr->dWo + (int64_t)b0 * d * d; a.ldd = d; a.d_sb = d * d;
    run_gemm(a);
    float* outs[3] = {gr->dWq, gr->dWk, gr->dWv};
    for (int w = 0; w < 3; ++w) {  // dWq = dQ^T y, ...
      GemmArgs b = base_args();
      b.M = (int)d; b.N = (int)d; b.K = (int)N; b.batch = nb;
      b.A = at(c->dQKV, (int64_t)b0 * 3 * state + (int64_t)w * d); b.a_sm = 1; b.a_sk = 3 * d; b.a_sb = 3 * state;
      b.B = at(c->Y, (int64_t)(2 * b0) * state); b.b_sn = 1; b.b_sk = d; b.b_sb = 2 * state;
      b.epi = EPI_STORE; b.d_f32 = true;
      b.D = outs[w] + (int64_t)b0 * d * d; b.ldd = d; b.d_sb = d * d;
      run_gemm(b);
    }
  }

  // ---- RNN ---------------------------------------------------------------------------------------
  // u_t = (g_{t+1} * tanh'(z_t)) W for every t at once (one GEMM over T*B rows)
  GemmArgs rnn_vjp_args() const {
    const int T = c->cfg.L;
    GemmArgs a = base_args();
    a.M = (int)(T * N); a.N = (int)d; a.K = (int)d;
    a.A = at(g, state); a.A2 = c->C; a.a_sm = d; a.a_sk = 1;
    a.B = p->W; a.b_sn = 1; a.b_sk = d;
    a.epi = EPI_STORE; a.D = c->U; a.ldd = d;
    if (c->cfg.loss == HBP_LOSS_EVERY_STEP) {  // u_t + delta_t in the epilogue: one tensor less for the scan
      a.epi = EPI_ADD; a.E = delta; a.lde = d;
    }
    if (c->Ahi) {  // float: g * tanh' split for the tf32 tensor-core product; B(n, k) = W[k][n] = W^T[n][k]
      a.A_hi = c->Ahi; a.A_lo = c->Alo;
      a.B_hi = c->Whi; a.B_lo = c->Wlo; a.hl_b_sn = d; a.hl_b_sk = 1;
    }
    return a;
  }
  void rnn_vjp_all() {
    const GemmArgs a = rnn_vjp_args();
    u_has_delta = a.epi == EPI_ADD;
    if (c->Ahi && !operand_ready)
      split_tf32(lc, (const float*)at(g, state), (const float*)c->C, c->Ahi, c->Alo, (int64_t)c->cfg.L * state);
    operand_ready = false;
    run_gemm(a);
  }
  // Whether the scan may write the split operand in place of the iterate: only if the tensor-core GEMM is going to
  // take the product (the CUDA-core kernel reads g itself).  Asked once per call: the answer depends on the
  // caller's pointers too.
  bool rnn_operand_from_scan() {
    if (rnn_tc < 0) {
      GemmArgs a = rnn_vjp_args();
      a.dry_run = true;
      rnn_tc = c->Ahi && c->scan_operand && !lc.force_simt && gemm_tc(lc, a, c->status) ? 1 : 0;
    }
    return rnn_tc == 1;
  }
  void rnn_wgrad(const hbp_grads* gr) {
    const int T = c->cfg.L;
    const int64_t rows = (int64_t)T * N, in = c->cfg.in_dim;
    // float on the tensor cores: at most 512 rows (16 k-blocks) per split keeps each fp32 accumulation chain
    // short; the partial sums are then added in double in a fixed order
    int split = (int)(rows / (c->Ahi ? 512 : 2048));
    if (split < 1) split = 1;
    if (split > kMaxSplit) split = kMaxSplit;
    for (int w = 0; w < 2; ++w) {
      GemmArgs a = base_args();  // dW = dZ^T H (H = states 0..T-1), dU = dZ^T X
      a.M = (int)d; a.N = w == 0 ? (int)d : (int)in; a.K = (int)rows;
      a.A = at(g, state); a.A2 = c->C; a.a_sm = 1; a.a_sk = d;
      a.B = w == 0 ? x_all : inputs; a.b_sn = 1; a.b_sk = a.N;
      if (c->Ahi) {  // tf32 path: transposed splits, so that the row index (the contraction) is contiguous
        if (w == 0)
          split_tf32_transposed(lc, (const float*)at(g, state), (const float*)c->C, c->Ahi, c->Alo, rows, (int)d);
        a.A_hi = c->Ahi; a.A_lo = c->Alo; a.hl_a_sm = rows; a.hl_a_sk = 1;
        a.B_hi = w == 0 ? c->Hhi : c->Xhi; a.B_lo = w == 0 ? c->Hlo : c->Xlo; a.hl_b_sn = rows; a.hl_b_sk = 1;
      }
      a.epi = EPI_STORE; a.d_f32 = true;
      a.D = w == 0 ? gr->dW : gr->dU; a.ldd = a.N;
      if (split > 1) { a.splitk = split; a.partial = c->partial; }
      if (a.D) run_gemm(a);
    }
  }

  // ---- GRU ---------------------------------------------------------------------------------------
  // u_t = (g_{t+1} * [c_r | c_z | c_nr]_t) W for every t at once: one GEMM over T*B rows with K = 3d
  void gru_vjp_all() {
    const int T = c->cfg.L;
    const int64_t rows = (int64_t)T * N;
    GemmArgs a = base_args();
    a.M = (int)rows; a.N = (int)d; a.K = (int)(3 * d);
    a.A = c->A4; a.a_sm = 4 * d; a.a_sk = 1;
    a.B = p->W; a.b_sn = 1; a.b_sk = d;
    a.epi = EPI_STORE; a.D = c->U; a.ldd = d;
    if (c->cfg.loss == HBP_LOSS_EVERY_STEP) {
      a.epi = EPI_ADD; a.E = delta; a.lde = d;
      u_has_delta = true;
    }
    bool tc = false;
    if (c->Ahi && !lc.force_simt) {
      gru_split(lc, (const float*)at(g, state), (const float*)c->C4, c->Ahi, c->Alo, rows, (int)d);
      a.A_hi = c->Ahi; a.A_lo = c->Alo; a.hl_a_sm = 3 * d; a.hl_a_sk = 1;
      a.B_hi = c->Whi; a.B_lo = c->Wlo; a.hl_b_sn = 3 * d; a.hl_b_sk = 1;
      tc = gemm_tc(lc, a, c->status);
    }
    if (!tc) {
      gru_operand(lc, c->cfg.dtype, at(g, state), c->C4, c->A4, rows, (int)d);
      a.A_hi = a.A_lo = a.B_hi = a.B_lo = nullptr;
      run_gemm(a);
    }
  }
  // dW = [dr|dz|d(W_n h)]^T H (H = states 0..T-1),  dU = [dr|dz|dn]^T X, with the pre-activation gradients
  // g * coefficients; dU is two products because its third row block uses another coefficient than dW's
  void gru_wgrad(const hbp_grads* gr) {
    const int T = c->cfg.L;
    const int64_t rows = (int64_t)T * N, in = c->cfg.in_dim;
    int split = (int)(rows / (c->Ahi ? 512 : 2048));
    if (split < 1) split = 1;
    if (split > kMaxSplit) split = kMaxSplit;
    const bool try_tc = c->Ahi && !lc.force_simt;
    if (try_tc) gru_split_transposed(lc, (const float*)at(g, state), (const float*)c->C4, c->Ahi, c->Alo, rows, (int)d);
    bool have_a4 = false;
    // {first row of the [4d] operand, rows, output, output row, against the states or the inputs}
    struct Part { int64_t a_row, m; float* out; int64_t out_row; bool states; };
    const Part parts[3] = {{0, 3 * d, gr->dW, 0, true}, {0, 2 * d, gr->dU, 0, false}, {3 * d, d, gr->dU, 2 * d, false}};
    for (const Part& pt : parts) {
      const int64_t n = pt.states ? d : in;
      GemmArgs a = base_args();
      a.M = (int)pt.m; a.N = (int)n; a.K = (int)rows;
      a.A = at(c->A4, pt.a_row); a.a_sm = 1; a.a_sk = 4 * d;
      a.B = pt.states ? x_all : inputs; a.b_sn = 1; a.b_sk = n;
      a.epi = EPI_STORE; a.d_f32 = true;
      a.D = pt.out + pt.out_row * n; a.ldd = n;
      if (split > 1) { a.splitk = split; a.partial = c->partial; }
      bool tc = false;
      if (try_tc) {
        a.A_hi = c->Ahi + pt.a_row * rows; a.A_lo = c->Alo + pt.a_row * rows; a.hl_a_sm = rows; a.hl_a_sk = 1;
        a.B_hi = pt.states ? c->Hhi : c->Xhi; a.B_lo = pt.states ? c->Hlo : c->Xlo; a.hl_b_sn = rows; a.hl_b_sk = 1;
        tc = gemm_tc(lc, a, c->status);
      }
      if (!tc) {
        if (!have_a4) gru_operand(lc, c->cfg.dtype, at(g, state), c->C4, c->A4, rows, (int)d);
        have_a4 = true;
        a.A_hi = a.A_lo = a.B_hi = a.B_lo = nullptr;
        run_gemm(a);
      }
    }
  }

  // ---- LSTM (u = d / 2 units; rows of g, U and the states are 2u wide) ------------------------------------
  // u_h = [t c_i | t c_f | t c_g | g_h c_o] W for every t at once (one GEMM, K = 4u); u_c elementwise beside it
  void lstm_vjp_all() {
    const int T = c->cfg.L;
    const int64_t rows = (int64_t)T * N, u = d / 2;
    const bool every = c->cfg.loss == HBP_LOSS_EVERY_STEP;
    GemmArgs a = base_args();
    a.M = (int)rows; a.N = (int)u; a.K = (int)(4 * u);
    a.A = c->A4; a.a_sm = 4 * u; a.a_sk = 1;
    a.B = p->W; a.b_sn = 1; a.b_sk = u;
    a.epi = EPI_STORE; a.D = at(c->U, u); a.ldd = d;
    if (every) {  // u_t + delta_t on both halves: the GEMM epilogue adds the h half, the operand kernels the c half
      a.epi = EPI_ADD; a.E = at(delta, u); a.lde = d;
      u_has_delta = true;
    }
    const void* dl = every ? delta : nullptr;
    bool tc = false;
    if (c->Ahi && !lc.force_simt) {
      lstm_split(lc, (const float*)at(g, state), (const float*)c->C5, (const float*)c->Fg, (const float*)dl, c->Ahi, c->Alo,
                 (float*)c->U, rows, (int)u);
      a.A_hi = c->Ahi; a.A_lo = c->Alo; a.hl_a_sm = 4 * u; a.hl_a_sk = 1;
      a.B_hi = c->Whi; a.B_lo = c->Wlo; a.hl_b_sn = 4 * u; a.hl_b_sk = 1;
      tc = gemm_tc(lc, a, c->status);
    }
    if (!tc) {
      lstm_operand(lc, c->cfg.dtype, at(g, state), c->C5, c->Fg, dl, c->A4, c->U, rows, (int)u);
      a.A_hi = a.A_lo = a.B_hi = a.B_lo = nullptr;
      run_gemm(a);
    }
  }
  // dW = [..]^T H (H = the h half of states 0..T-1), dU = [..]^T X with the same four-block operand
  void lstm_wgrad(const hbp_grads* gr) {
    const int T = c->cfg.L;
    const int64_t rows = (int64_t)T * N, in = c->cfg.in_dim, u = d / 2;
    int split = (int)(rows / (c->Ahi ? 512 : 2048));
    if (split < 1) split = 1;
    if (split > kMaxSplit) split = kMaxSplit;
    const bool try_tc = c->Ahi && !lc.force_simt;
    if (try_tc) lstm_split_transposed(lc, (const float*)at(g, state), (const float*)c->C5, c->Ahi, c->Alo, rows, (int)u);
    bool have_a4 = false;
    for (int w = 0; w < 2; ++w) {
      const int64_t n = w == 0 ? u : in;
      GemmArgs a = base_args();
      a.M = (int)(4 * u); a.N = (int)n; a.K = (int)rows;
      a.A = c->A4; a.a_sm = 1; a.a_sk = 4 * u;
      a.B = w == 0 ? at(x_all, u) : inputs; a.b_sn = 1; a.b_sk = w == 0 ? d : in;
      a.epi = EPI_STORE; a.d_f32 = true;
      a.D = w == 0 ? gr->dW : gr->dU; a.ldd = n;
      if (split > 1) { a.splitk = split; a.partial = c->partial; }
      bool tc = false;
      if (try_tc) {
        a.A_hi = c->Ahi; a.A_lo = c->Alo; a.hl_a_sm = rows; a.hl_a_sk = 1;
        a.B_hi = w == 0 ? c->Hhi : c->Xhi; a.B_lo = w == 0 ? c->Hlo : c->Xlo; a.hl_b_sn = rows; a.hl_b_sk = 1;
        tc = gemm_tc(lc, a, c->status);
      }
      if (!tc) {
        if (!have_a4) lstm_operand(lc, c->cfg.dtype, at(g, state), c->C5, c->Fg, nullptr, c->A4, nullptr, rows, (int)u);
        have_a4 = true;
        a.A_hi = a.A_lo = a.B_hi = a.B_lo = nullptr;
        run_gemm(a);
      }
    }
  }

  // ---- all kinds: Eq. 8 for every step at once, and the parameter pass of Section 4.2 ---------------------------
  void vjp_all() {
    const int layers = c->layers, grp = c->group;
    switch (c->cfg.block) {
      case HBP_BLOCK_RNN_TANH: rnn_vjp_all(); break;
      case HBP_BLOCK_GRU: gru_vjp_all(); break;
      case HBP_BLOCK_LSTM: lstm_vjp_all(); break;
      default:
        mask_gradients(0, layers);
        for (int b0 = 0; b0 < layers; b0 += grp) mlp_vjp(b0, b0 + grp < layers ? b0 + grp : layers, true);
        if (c->cfg.block == HBP_BLOCK_PRELN_TRANSFORMER) attn_vjp(0, layers, true);
    }
  }
  void wgrad_all(const hbp_grads* gr) {
    const int layers = c->layers, grp = c->group;
    switch (c->cfg.block) {
      case HBP_BLOCK_RNN_TANH: rnn_wgrad(gr); break;
      case HBP_BLOCK_GRU: gru_wgrad(gr); break;
      case HBP_BLOCK_LSTM: lstm_wgrad(gr); break;
      default:
        mask_gradients(0, layers);
        for (int b0 = 0; b0 < layers; b0 += grp) {
          const int b1 = b0 + grp < layers ? b0 + grp : layers;
          mlp_vjp(b0, b1, false);
          mlp_wgrad(b0, b1, gr);
        }
        if (c->cfg.block == HBP_BLOCK_PRELN_TRANSFORMER) {
          attn_vjp(0, layers, false);
          attn_wgrad(0, layers, gr);
        }
    }
    gate_grads(gr);
  }

  void gate_grads(const hbp_grads* gr) {
    if (!gr->da || c->cfg.gate == HBP_GATE_ONE) return;
    if (c->cfg.gate == HBP_GATE_CHANNEL_SHARED) {
      gate_grad(lc, c->cfg.dtype, at(g, state), x_all, (int64_t)c->steps * N, (int)d, gr->da, c->partial, kGateBlocks);
    } else {
      for (int l = 0; l < c->steps; ++l)
        gate_grad(lc, c->cfg.dtype, at(g, (int64_t)(l + 1) * state), at(x_all, (int64_t)l * state), N, (int)d,
                  gr->da + (int64_t)l * d, c->partial, kGateBlocks);
    }
  }

  // Reverse scan over steps [lo, hi) that adds the block VJPs in U (finishing LayerNorm-backward on the way).
  void scan_with_u(int lo, int hi) {
    if (c->preln && c->lnpart && stats_ok)
      ln_stats_finish(lc, c->lnpart + (int64_t)lo * N * c->ln_slots, c->ln_slots, c->rstd + (int64_t)lo * N,
                      c->lnstat + (int64_t)lo * N, (int64_t)(hi - lo) * N, (int)d);
    scan_reverse(lc, scan_args(lo, hi, true));
    stats_ok = true;
  }
  ScanArgs scan_args(int lo, int hi, bool with_u) const {
    ScanArgs s;
    s.dtype = c->cfg.dtype; s.L = c->steps; s.l_lo = lo; s.l_hi = hi; s.rows = N; s.d = (int)d;
    s.u = with_u ? c->U : nullptr;
    s.u_has_delta = with_u && u_has_delta;
    if (shifted) {
      s.keep = 1.0f - c->cfg.gamma;
      s.gamma = with_u ? c->cfg.gamma : 0.0f;
    }
    s.delta = delta; s.loss = c->cfg.loss;
    s.a = p->a; s.gate = c->cfg.gate;
    if (c->cfg.block == HBP_BLOCK_GRU) { s.a = c->Zc; s.gate = kGateElement; }
    if (c->cfg.block == HBP_BLOCK_LSTM) { s.a = c->Fg; s.gate = kGateElement; }
    if (c->cfg.block == HBP_BLOCK_RELU_MLP) { s.a = c->MASK; s.gate = kGateElement; }
    if (c->cfg.block == HBP_BLOCK_POSTLN_MLP) {
      s.gate = kGateRow; s.row_gate = c->rstd;
      if (with_u) s.u2 = c->CB;
    }
    s.g = g;
    if (want_operand && !shifted && lo == 0 && hi == c->steps) {
      s.op_coef = (const float*)c->C; s.op_hi = c->Ahi; s.op_lo = c->Alo;
      s.op_skip_g = true;  // an intermediate iterate: only its product with the coefficients is read
      s.op_done = &operand_ready;
    }
    if (with_u && c->preln) {
      s.xhat = c->Y; s.rstd = c->rstd;
      if (c->lnpart && stats_ok) s.lnstat = c->lnstat;
    }
    s.scratch = c->scan_scratch; s.scratch_bytes = c->scan_scratch_bytes;
    s.status = c->status;
    return s;
  }
  void set_last_state() {
    const char* dl = c->cfg.loss == HBP_LOSS_EVERY_STEP ? at(delta, (int64_t)c->steps * state) : delta;
    copy_state(lc, c->cfg.dtype, at(g, (int64_t)c->steps * state), dl, state);
  }
};

// Records a pair of events around one phase of a call while profiling is on.
struct PhaseScope {
  hbp_ctx* c;
  cudaStream_t stream;
  ProfSeg seg;
  bool live = false;
  int64_t launches0 = 0;
  PhaseScope(Run& r, int phase) : c(r.c), stream(r.lc.stream) {
    if (!c->profiling || c->segs.size() >= 8192) return;
    if (!c->free_segs.empty()) {
      seg = c->free_segs.back();
      c->free_segs.pop_back();
    } else if (cudaEventCreate(&seg.beg) != cudaSuccess || cudaEventCreate(&seg.end) != cudaSuccess) {
      return;
    }
    seg.phase = phase;
    launches0 = c->launches;
    live = cudaEventRecord(seg.beg, stream) == cudaSuccess;
  }
  ~PhaseScope() {
    if (!live) return;
    cudaEventRecord(seg.end, stream);
    seg.launches = c->launches - launches0;
    c->segs.push_back(seg);
  }
};

hbp_status check_call(hbp_ctx* ctx, const hbp_params* p, bool need_forward) {
  if (!ctx || !p) return HBP_ERR_INVALID_ARG;
  if (need_forward && !ctx->forward_done) return HBP_ERR_STATE;
  const hbp_config& f = ctx->cfg;
  if (f.block == HBP_BLOCK_RNN_TANH || f.block == HBP_BLOCK_GRU || f.block == HBP_BLOCK_LSTM) {
    if (!p->W || !p->U) return HBP_ERR_INVALID_ARG;
  } else {
    if (!p->W1 || !p->W2) return HBP_ERR_INVALID_ARG;
    if (f.block == HBP_BLOCK_PRELN_TRANSFORMER && (!p->Wq || !p->Wk || !p->Wv || !p->Wo)) return HBP_ERR_INVALID_ARG;
  }
  if (f.gate != HBP_GATE_ONE && !p->a) return HBP_ERR_INVALID_ARG;
  return HBP_OK;
}

hbp_status check_grads(const hbp_ctx* ctx, const hbp_grads* g) {
  if (!g) return HBP_OK;
  const hbp_config& f = ctx->cfg;
  if (f.block == HBP_BLOCK_RNN_TANH || f.block == HBP_BLOCK_GRU || f.block == HBP_BLOCK_LSTM) return (g->dW && g->dU) ? HBP_OK : HBP_ERR_INVALID_ARG;
  if (!g->dW1 || !g->dW2) return HBP_ERR_INVALID_ARG;
  if (f.block == HBP_BLOCK_PRELN_TRANSFORMER && (!g->dWq || !g->dWk || !g->dWv || !g->dWo)) return HBP_ERR_INVALID_ARG;
  return HBP_OK;
}

bool misaligned(const void* p) { return ((uintptr_t)p & 15u) != 0; }

}  // namespace

extern "C" {

const char* hbp_status_string(hbp_status s) {
  switch (s) {
    case HBP_OK: return "ok";
    case HBP_ERR_INVALID_ARG: return "invalid argument";
    case HBP_ERR_SHAPE: return "bad shape or alignment";
    case HBP_ERR_DTYPE: return "bad dtype";
    case HBP_ERR_STATE: return "backward before forward";
    case HBP_ERR_WORKSPACE: return "workspace too small or misaligned";
    case HBP_ERR_UNSUPPORTED: return "unsupported configuration";
    case HBP_ERR_CUDA: return "CUDA error";
    case HBP_ERR_TIMEOUT: return "bounded device wait expired";
  }
  return "unknown status";
}

hbp_status hbp_workspace_bytes(const hbp_config* cfg, size_t* bytes) {
  if (!bytes) return HBP_ERR_INVALID_ARG;
  hbp_status st = check_config(cfg);
  if (st != HBP_OK) return st;
  hbp_ctx tmp;
  tmp.cfg = *cfg;
  *bytes = carve(&tmp, nullptr);
  return HBP_OK;
}

hbp_status hbp_create(const hbp_config* cfg, void* workspace, size_t workspace_bytes, hbp_ctx** out) {
  if (!out) return HBP_ERR_INVALID_ARG;
  *out = nullptr;
  hbp_status st = check_config(cfg);
  if (st != HBP_OK) return st;
  if (!workspace || ((uintptr_t)workspace % kAlign)) return HBP_ERR_WORKSPACE;
  hbp_ctx* c = new (std::nothrow) hbp_ctx;
  if (!c) return HBP_ERR_INVALID_ARG;
  c->cfg = *cfg;
  const size_t need = carve(c, (char*)workspace);
  if (workspace_bytes < need) {
    delete c;
    return HBP_ERR_WORKSPACE;
  }
  c->ws = (char*)workspace;
  c->ws_bytes = workspace_bytes;
  const char* env = std::getenv("HBP_FORCE_SIMT");
  c->force_simt = env && env[0] == '1';
  const char* pm = std::getenv("HBP_GEMM_PAIR");
  c->gemm_pair = !(pm && pm[0] == '0');  // pairs by default
  const char* so = std::getenv("HBP_SCAN_OPERAND");
  c->scan_operand = !(so && so[0] == '0');  // the scan writes the next VJP's operand by default (float tanh RNN)
  if (cudaMemset(c->status, 0, 256) != cudaSuccess) {
    delete c;
    return HBP_ERR_CUDA;
  }
  *out = c;
  return HBP_OK;
}

void hbp_destroy(hbp_ctx* ctx) {
  if (!ctx) return;
  for (auto* v : {&ctx->segs, &ctx->free_segs})
    for (ProfSeg& s : *v) {
      cudaEventDestroy(s.beg);
      cudaEventDestroy(s.end);
    }
  delete ctx;
}

hbp_status hbp_profile_enable(hbp_ctx* ctx, int32_t on) {
  if (!ctx) return HBP_ERR_INVALID_ARG;
  ctx->profiling = on != 0;
  for (ProfSeg& s : ctx->segs) ctx->free_segs.push_back(s);
  ctx->segs.clear();
  return HBP_OK;
}

hbp_status hbp_profile_read(hbp_ctx* ctx, float* ms, int64_t* launches) {
  if (!ctx) return HBP_ERR_INVALID_ARG;
  float t[HBP_PHASE_COUNT] = {0, 0, 0, 0};
  int64_t n[HBP_PHASE_COUNT] = {0, 0, 0, 0};
  hbp_status st = HBP_OK;
  for (ProfSeg& s : ctx->segs) {
    float e = 0.0f;
    if (cudaEventSynchronize(s.end) != cudaSuccess || cudaEventElapsedTime(&e, s.beg, s.end) != cudaSuccess) st = HBP_ERR_CUDA;
    t[s.phase] += e;
    n[s.phase] += s.launches;
    ctx->free_segs.push_back(s);
  }
  ctx->segs.clear();
  for (int i = 0; i < HBP_PHASE_COUNT; ++i) {
    if (ms) ms[i] = t[i];
    if (launches) launches[i] = n[i];
  }
  return st;
}

int64_t hbp_launch_count(const hbp_ctx* ctx) { return ctx ? ctx->launches : 0; }

int32_t hbp_context_modes(const hbp_ctx* ctx) { return ctx ? (ctx->force_simt ? 1 : 0) | (ctx->gemm_pair ? 2 : 0) | (ctx->scan_operand ? 4 : 0) : 0; }

hbp_status hbp_sync_status(hbp_ctx* ctx, void* cuda_stream) {
  if (!ctx) return HBP_ERR_INVALID_ARG;
  int word = 0;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  if (cudaMemcpyAsync(&word, ctx->status, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return HBP_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return HBP_ERR_CUDA;
  if (word != 0) {  // reported once: the next calls start from a clean word
    if (cudaMemsetAsync(ctx->status, 0, sizeof(int), s) != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess) return HBP_ERR_CUDA;
  }
  return (hbp_status)word;
}

hbp_status hbp_selftest_wait_timeout(hbp_ctx* ctx, void* scratch, size_t scratch_bytes, uint64_t limit_ns, void* cuda_stream) {
  if (!ctx || !scratch) return HBP_ERR_INVALID_ARG;
  if (((uintptr_t)scratch % kAlign) || scratch_bytes < ((size_t)128 << 10)) return HBP_ERR_WORKSPACE;
  if (limit_ns < 1000 || limit_ns > 1000000000ull) return HBP_ERR_INVALID_ARG;
  Launcher lc;
  lc.stream = (cudaStream_t)cuda_stream;
  lc.launches = &ctx->launches;
  // one 128 x 256 x 64 bf16 tile; the producer arms the first pipeline stage and issues no copy, so the MMA role's
  // wait for it runs out after limit_ns
  char* base = (char*)scratch;
  GemmArgs g;
  g.in_dtype = HBP_BF16;
  g.M = 128; g.N = 256; g.K = 64;
  g.A = base; g.a_sm = 64; g.a_sk = 1;
  g.B = base + (16 << 10); g.b_sn = 64; g.b_sk = 1;
  g.epi = EPI_STORE;
  g.D = base + (48 << 10); g.ldd = 256;
  g.wait_limit_ns = limit_ns;
  g.test_stall = 1;
  if (!gemm_tc(lc, g, ctx->status)) return HBP_ERR_UNSUPPORTED;
  return lc.err == cudaSuccess ? HBP_OK : HBP_ERR_CUDA;
}

hbp_status hbp_forward(hbp_ctx* ctx, const hbp_params* params, const void* x0, const void* inputs, void* x_all,
                       void* cuda_stream) {
  hbp_status st = check_call(ctx, params, false);
  if (st != HBP_OK) return st;
  if (!x0 || !x_all) return HBP_ERR_INVALID_ARG;
  if (misaligned(x0) || misaligned(x_all)) return HBP_ERR_SHAPE;
  const hbp_config& f = ctx->cfg;
  if ((f.block == HBP_BLOCK_RNN_TANH || f.block == HBP_BLOCK_GRU || f.block == HBP_BLOCK_LSTM) && !inputs) return HBP_ERR_INVALID_ARG;
  Run r(ctx, params, cuda_stream);
  r.x_all = (const char*)x_all;
  char* xa = (char*)x_all;
  const int64_t N = r.N, d = r.d, h = r.h, state = r.state;
  copy_state(r.lc, f.dtype, xa, x0, state);
  if (ctx->xres) convert_to_f32(r.lc, f.dtype, x0, ctx->xres, state);

  if (f.block == HBP_BLOCK_LSTM) {
    const int T = f.L;
    const int64_t u = d / 2;
    convert_to_f64(r.lc, f.dtype, x0, ctx->hres, state);
    for (int t = 0; t < T; ++t) {
      const double* sin = ctx->hres + (int64_t)(t & 1) * state;
      double* sout = ctx->hres + (int64_t)((t + 1) & 1) * state;
      lstm_forward_step(r.lc, f.dtype, params->W, params->U, r.at(inputs, (int64_t)t * N * f.in_dim), sin, sout,
                        r.at(ctx->Fg, (int64_t)t * state), r.at(ctx->C5, (int64_t)t * N * 5 * u),
                        r.at(xa, (int64_t)(t + 1) * state), (int)N, (int)u, f.in_dim);
    }
    if (ctx->Ahi) {
      split_tf32_transposed(r.lc, (const float*)xa + u, nullptr, ctx->Hhi, ctx->Hlo, (int64_t)T * N, (int)u, d);
      split_tf32_transposed(r.lc, (const float*)inputs, nullptr, ctx->Xhi, ctx->Xlo, (int64_t)T * N, f.in_dim);
      split_tf32_transposed(r.lc, (const float*)params->W, nullptr, ctx->Whi, ctx->Wlo, 4 * u, (int)u);  // -> [u][4u]
    }
  } else if (f.block == HBP_BLOCK_GRU) {
    const int T = f.L;
    convert_to_f64(r.lc, f.dtype, x0, ctx->hres, state);
    for (int t = 0; t < T; ++t) {
      const double* hin = ctx->hres + (int64_t)(t & 1) * state;
      double* hout = ctx->hres + (int64_t)((t + 1) & 1) * state;
      gru_forward_step(r.lc, f.dtype, params->W, params->U, r.at(inputs, (int64_t)t * N * f.in_dim), hin, hout,
                       r.at(ctx->Zc, (int64_t)t * state), r.at(ctx->C4, (int64_t)t * 4 * state),
                       r.at(xa, (int64_t)(t + 1) * state), (int)N, (int)d, f.in_dim);
    }
    if (ctx->Ahi) {
      split_tf32_transposed(r.lc, (const float*)xa, nullptr, ctx->Hhi, ctx->Hlo, (int64_t)T * N, (int)d);
      split_tf32_transposed(r.lc, (const float*)inputs, nullptr, ctx->Xhi, ctx->Xlo, (int64_t)T * N, f.in_dim);
      split_tf32_transposed(r.lc, (const float*)params->W, nullptr, ctx->Whi, ctx->Wlo, 3 * d, (int)d);  // -> [d][3d]
    }
  } else if (f.block == HBP_BLOCK_RNN_TANH) {
    const int T = f.L;
    // all T steps in one launch where that form applies, else one launch per step
    const bool one_launch = ctx->Pd && !ctx->force_simt &&
                            rnn_forward_persistent(r.lc, f.dtype, params->W, params->U, inputs, r.gate_ptr(0), x0, ctx->Pd, xa,
                                                   ctx->C, T, (int)N, (int)d, f.in_dim, ctx->status);
    if (!one_launch) {
      convert_to_f64(r.lc, f.dtype, x0, ctx->hres, state);
      for (int t = 0; t < T; ++t) {
        const double* hin = ctx->hres + (int64_t)(t & 1) * state;
        double* hout = ctx->hres + (int64_t)((t + 1) & 1) * state;
        rnn_forward_step(r.lc, f.dtype, params->W, params->U, r.at(inputs, (int64_t)t * N * f.in_dim), r.gate_ptr(t), hin,
                         hout, r.at(ctx->C, (int64_t)t * state), r.at(xa, (int64_t)(t + 1) * state), (int)N, (int)d,
                         f.in_dim);
      }
    }
    if (ctx->Ahi) {  // operand splits that do not change between backward calls
      split_tf32_transposed(r.lc, (const float*)xa, nullptr, ctx->Hhi, ctx->Hlo, (int64_t)T * N, (int)d);
      split_tf32_transposed(r.lc, (const float*)inputs, nullptr, ctx->Xhi, ctx->Xlo, (int64_t)T * N, f.in_dim);
      split_tf32_transposed(r.lc, (const float*)params->W, nullptr, ctx->Whi, ctx->Wlo, d, (int)d);
    }
  } else {
    const bool tr = f.block == HBP_BLOCK_PRELN_TRANSFORMER;
    if (tr) {  // stack Wq, Wk, Wv per layer so that QKV and its VJP are single GEMMs
      const size_t blk = (size_t)d * d * r.es;
      const void* src[3] = {params->Wq, params->Wk, params->Wv};
      for (int w = 0; w < 3; ++w) {
        cudaError_t e = cudaMemcpy2DAsync(ctx->Wqkv + w * blk, 3 * blk, src[w], blk, blk, (size_t)f.L,
                                          cudaMemcpyDeviceToDevice, r.lc.stream);
        if (e != cudaSuccess && r.lc.err == cudaSuccess) r.lc.err = e;
      }
    }
    // residual update x_{l+1} = a * x_l + F through the float master copy when there is one
    auto resid_epilogue = [&](GemmArgs& a, int step) {
      a.epi = EPI_RESID;
      a.gate = r.gate_ptr(step);
      if (ctx->xres) a.R = ctx->xres;
      else { a.E = r.at(xa, (int64_t)step * state); a.lde = d; }
      a.D = r.at(xa, (int64_t)(step + 1) * state); a.ldd = d;
      if (ctx->MASK) { a.relu = true; a.D2 = r.at(ctx->MASK, (int64_t)step * state); a.ldd2 = d; }
    };
    auto ln_of = [&](int step) {
      const void* src = ctx->xres ? (const void*)ctx->xres : (const void*)r.at(xa, (int64_t)step * state);
      layernorm_fwd(r.lc, f.dtype, src, ctx->xres != nullptr, r.at(ctx->Y, (int64_t)step * state),
                    ctx->rstd + (int64_t)step * N, N, (int)d, f.ln_eps);
    };
    for (int b = 0; b < f.L; ++b) {
      if (tr) {
        const int step = 2 * b;
        ln_of(step);
        GemmArgs q = r.base_args();
        q.M = (int)N; q.N = (int)(3 * d); q.K = (int)d;
        q.A = r.at(ctx->Y, (int64_t)step * state); q.a_sm = d; q.a_sk = 1;
        q.B = r.at(ctx->Wqkv, (int64_t)b * 3 * d * d); q.b_sn = d; q.b_sk = 1;
        q.epi = EPI_STORE; q.D = r.at(ctx->QKV, (int64_t)b * 3 * state); q.ldd = 3 * d;
        r.run_gemm(q);
        AttnArgs t;
        t.dtype = f.dtype; t.batch = f.batch; t.seq = f.seq; t.heads = f.n_heads; t.head_dim = f.head_dim;
        t.qkv = r.at(ctx->QKV, (int64_t)b * 3 * state);
        t.o = r.at(ctx->O, (int64_t)b * state);
        t.lse = ctx->lse + (int64_t)b * f.batch * f.n_heads * f.seq;
        t.status = ctx->status;
        attention_fwd(r.lc, t);
        GemmArgs o = r.base_args();
        o.M = (int)N; o.N = (int)d; o.K = (int)d;
        o.A = r.at(ctx->O, (int64_t)b * state); o.a_sm = d; o.a_sk = 1;
        o.B = r.at(params->Wo, (int64_t)b * d * d); o.b_sn = d; o.b_sk = 1;
        resid_epilogue(o, step);
        r.run_gemm(o);
      }
      const int step = r.mlp_step(b);
      if (ctx->preln) ln_of(step);
      GemmArgs a = r.base_args();
      a.M = (int)N; a.N = (int)h; a.K = (int)d;
      a.A = r.mlp_operand(b); a.a_sm = d; a.a_sk = 1;
      a.B = r.at(params->W1, (int64_t)b * h * d); a.b_sn = d; a.b_sk = 1;
      a.epi = EPI_GELU_FWD;
      a.D = r.at(ctx->ACT, (int64_t)b * N * h); a.ldd = h;
      a.D2 = r.at(ctx->DACT, (int64_t)b * N * h); a.ldd2 = h;
      r.run_gemm(a);
      GemmArgs c2 = r.base_args();
      c2.M = (int)N; c2.N = (int)d; c2.K = (int)h;
      c2.A = r.at(ctx->ACT, (int64_t)b * N * h); c2.a_sm = h; c2.a_sk = 1;
      c2.B = r.at(params->W2, (int64_t)b * d * h); c2.b_sn = h; c2.b_sk = 1;
      resid_epilogue(c2, step);
      r.run_gemm(c2);
      if (f.block == HBP_BLOCK_POSTLN_MLP) {  // x_{l+1} = LN(x_l + Block(x_l)), normalised in place; 1/sigma is the gate
        const void* src = ctx->xres ? (const void*)ctx->xres : (const void*)r.at(xa, (int64_t)(step + 1) * state);
        layernorm_fwd(r.lc, f.dtype, src, ctx->xres != nullptr, r.at(xa, (int64_t)(step + 1) * state),
                      ctx->rstd + (int64_t)step * N, N, (int)d, f.ln_eps, ctx->xres);
      }
    }
  }
  ctx->forward_done = true;
  return r.result();
}

static hbp_status backward_common(hbp_ctx* ctx, const hbp_params* params, int32_t k, bool exact, const void* delta,
                                  const void* x_all, const void* inputs, void* g_all, const hbp_grads* grads,
                                  void* cuda_stream) {
  hbp_status st = check_call(ctx, params, true);
  if (st != HBP_OK) return st;
  if (!delta || !x_all || !g_all || k < 0) return HBP_ERR_INVALID_ARG;
  if (misaligned(delta) || misaligned(x_all) || misaligned(g_all)) return HBP_ERR_SHAPE;
  st = check_grads(ctx, grads);
  if (st != HBP_OK) return st;
  const hbp_config& f = ctx->cfg;
  if ((f.block == HBP_BLOCK_RNN_TANH || f.block == HBP_BLOCK_GRU || f.block == HBP_BLOCK_LSTM) && grads && !inputs) return HBP_ERR_INVALID_ARG;
  Run r(ctx, params, cuda_stream);
  r.x_all = (const char*)x_all;
  r.inputs = (const char*)inputs;
  r.g = (char*)g_all;
  r.delta = (const char*)delta;
  const int steps = ctx->steps;
  const bool tr = f.block == HBP_BLOCK_PRELN_TRANSFORMER, rnn = f.block == HBP_BLOCK_RNN_TANH;
  const bool gru = f.block == HBP_BLOCK_GRU;
  {
    PhaseScope ph(r, HBP_PHASE_OTHER);
    r.set_last_state();
  }

  if (!exact) {
    r.shifted = f.gamma != 0.0f;
    // g^0 = CumSumProd(delta, K) (Eq. 10), then k iterations of {all-step VJP (Eq. 8); reverse scan (Eq. 9, 11)}
    const int iters = k < steps ? k : steps;
    {
      PhaseScope ph(r, HBP_PHASE_OTHER);  // g^0: a scan without VJPs (a broadcast of delta_L when a = 1)
      r.want_operand = rnn && iters > 0 && r.rnn_operand_from_scan();
      scan_reverse(r.lc, r.scan_args(0, steps, false));
    }
    for (int it = 0; it < iters; ++it) {
      {
        PhaseScope ph(r, HBP_PHASE_VJP);
        r.vjp_all();
      }
      PhaseScope ph(r, HBP_PHASE_SCAN);
      r.want_operand = rnn && it + 1 < iters && r.rnn_operand_from_scan();
      r.scan_with_u(0, steps);
    }
    r.want_operand = false;
    if (grads) {  // Section 4.2: parameter gradients from the final estimate
      PhaseScope ph(r, HBP_PHASE_WGRAD);
      r.wgrad_all(grads);
    }
  } else {
    // Section 2.2: g_l = delta_l + a_l g_{l+1} + J_l^T g_{l+1}, one step at a time
    PhaseScope ph(r, HBP_PHASE_OTHER);
    if (rnn) {
      // the sequential recurrence is carried in double beside the stored float gradients: one launch over all
      // steps where that form applies, else one launch per step
      const bool one_launch = ctx->Pd && !ctx->force_simt &&
                              rnn_backward_persistent(r.lc, f.dtype, params->W, r.gate_ptr(0), ctx->C,
                                                      f.loss == HBP_LOSS_EVERY_STEP ? r.delta : nullptr, r.g, steps,
                                                      (int)r.N, (int)r.d, ctx->status);
      if (!one_launch) {
        convert_to_f64(r.lc, f.dtype, r.at(r.g, (int64_t)steps * r.state), ctx->hres, r.state);
        for (int t = steps - 1; t >= 0; --t) {
          const double* gin = ctx->hres + (int64_t)((steps - 1 - t) & 1) * r.state;
          double* gout = ctx->hres + (int64_t)((steps - t) & 1) * r.state;
          rnn_backward_step(r.lc, f.dtype, params->W, r.at(ctx->C, (int64_t)t * r.state),
                            f.loss == HBP_LOSS_EVERY_STEP ? r.at(r.delta, (int64_t)t * r.state) : nullptr, r.gate_ptr(t),
                            gin, gout, r.at(r.g, (int64_t)t * r.state), (int)r.N, (int)r.d);
        }
      }
      if (grads) r.rnn_wgrad(grads);
    } else if (gru) {
      convert_to_f64(r.lc, f.dtype, r.at(r.g, (int64_t)steps * r.state), ctx->hres, r.state);
      for (int t = steps - 1; t >= 0; --t) {
        const double* gin = ctx->hres + (int64_t)((steps - 1 - t) & 1) * r.state;
        double* gout = ctx->hres + (int64_t)((steps - t) & 1) * r.state;
        gru_backward_step(r.lc, f.dtype, params->W, r.at(ctx->Zc, (int64_t)t * r.state),
                          r.at(ctx->C4, (int64_t)t * 4 * r.state),
                          f.loss == HBP_LOSS_EVERY_STEP ? r.at(r.delta, (int64_t)t * r.state) : nullptr, gin, gout,
                          r.at(r.g, (int64_t)t * r.state), (int)r.N, (int)r.d);
      }
      if (grads) r.gru_wgrad(grads);
    } else if (f.block == HBP_BLOCK_LSTM) {
      convert_to_f64(r.lc, f.dtype, r.at(r.g, (int64_t)steps * r.state), ctx->hres, r.state);
      for (int t = steps - 1; t >= 0; --t) {
        const double* gin = ctx->hres + (int64_t)((steps - 1 - t) & 1) * r.state;
        double* gout = ctx->hres + (int64_t)((steps - t) & 1) * r.state;
        lstm_backward_step(r.lc, f.dtype, params->W, r.at(ctx->Fg, (int64_t)t * r.state),
                           r.at(ctx->C5, (int64_t)t * r.N * 5 * (r.d / 2)),
                           f.loss == HBP_LOSS_EVERY_STEP ? r.at(r.delta, (int64_t)t * r.state) : nullptr, gin, gout,
                           r.at(r.g, (int64_t)t * r.state), (int)r.N, (int)(r.d / 2));
      }
      if (grads) r.lstm_wgrad(grads);
    } else {
      for (int l = steps - 1; l >= 0; --l) {
        const int b = tr ? l / 2 : l;
        const bool is_mlp = !tr || (l % 2 == 1);
        if (is_mlp) {
          r.mask_gradients(b, b + 1);
          r.mlp_vjp(b, b + 1, true);
          if (grads) r.mlp_wgrad(b, b + 1, grads);
        } else {
          r.attn_vjp(b, b + 1, true);
          if (grads) r.attn_wgrad(b, b + 1, grads);
        }
        r.scan_with_u(l, l + 1);
      }
    }
    if (grads) r.gate_grads(grads);
  }
  return r.result();
}

hbp_status hbp_backward(hbp_ctx* ctx, const hbp_params* params, int32_t k, const void* delta, const void* x_all,
                        const void* inputs, void* g_all, const hbp_grads* grads, void* cuda_stream) {
  return backward_common(ctx, params, k, false, delta, x_all, inputs, g_all, grads, cuda_stream);
}

hbp_status hbp_exact(hbp_ctx* ctx, const hbp_params* params, const void* delta, const void* x_all, const void* inputs,
                     void* g_all, const hbp_grads* grads, void* cuda_stream) {
  return backward_common(ctx, params, 0, true, delta, x_all, inputs, g_all, grads, cuda_stream);
}

hbp_status hbp_iterate(hbp_ctx* ctx, const hbp_params* params, const void* delta, const void* x_all, const void* inputs,
                       void* g_all, void* cuda_stream) {
  hbp_status st = check_call(ctx, params, true);
  if (st != HBP_OK) return st;
  if (!delta || !x_all || !g_all) return HBP_ERR_INVALID_ARG;
  if (misaligned(delta) || misaligned(x_all) || misaligned(g_all)) return HBP_ERR_SHAPE;
  Run r(ctx, params, cuda_stream);
  r.x_all = (const char*)x_all;
  r.inputs = (const char*)inputs;
  r.g = (char*)g_all;
  r.delta = (const char*)delta;
  r.shifted = ctx->cfg.gamma != 0.0f;
  {
    PhaseScope ph(r, HBP_PHASE_VJP);
    r.vjp_all();  // from the iterate as given, g_all[steps] included
  }
  PhaseScope ph(r, HBP_PHASE_SCAN);
  r.set_last_state();
  r.scan_with_u(0, ctx->steps);
  return r.result();
}

hbp_status hbp_param_grads(hbp_ctx* ctx, const hbp_params* params, const void* x_all, const void* inputs, const void* g_all,
                           const hbp_grads* grads, void* cuda_stream) {
  hbp_status st = check_call(ctx, params, true);
  if (st != HBP_OK) return st;
  if (!x_all || !g_all || !grads) return HBP_ERR_INVALID_ARG;
  if (misaligned(x_all) || misaligned(g_all)) return HBP_ERR_SHAPE;
  st = check_grads(ctx, grads);
  if (st != HBP_OK) return st;
  const hbp_config& f = ctx->cfg;
  if ((f.block == HBP_BLOCK_RNN_TANH || f.block == HBP_BLOCK_GRU || f.block == HBP_BLOCK_LSTM) && !inputs) return HBP_ERR_INVALID_ARG;
  Run r(ctx, params, cuda_stream);
  r.x_all = (const char*)x_all;
  r.inputs = (const char*)inputs;
  r.g = (char*)const_cast<void*>(g_all);  // read only by the parameter pass
  PhaseScope ph(r, HBP_PHASE_WGRAD);
  r.wgrad_all(grads);
  return r.result();
}

hbp_status hbp_add_carry(hbp_ctx* ctx, const void* carry, void* g_all, void* cuda_stream) {
  if (!ctx || !carry || !g_all) return HBP_ERR_INVALID_ARG;
  if (misaligned(carry) || misaligned(g_all)) return HBP_ERR_SHAPE;
  if (ctx->cfg.gate != HBP_GATE_ONE || ctx->cfg.gamma != 0.0f || ctx->cfg.block == HBP_BLOCK_GRU ||
      ctx->cfg.block == HBP_BLOCK_LSTM || ctx->cfg.block == HBP_BLOCK_RELU_MLP ||
      ctx->cfg.block == HBP_BLOCK_POSTLN_MLP)
    return HBP_ERR_UNSUPPORTED;
  Launcher lc;
  lc.stream = (cudaStream_t)cuda_stream;
  lc.launches = &ctx->launches;
  add_to_states(lc, ctx->cfg.dtype, g_all, carry, ctx->steps + 1, (int64_t)ctx->cfg.tokens * ctx->cfg.d);
  return lc.err == cudaSuccess ? HBP_OK : HBP_ERR_CUDA;
}

size_t hbp_compare_scratch_bytes(int32_t segments) { return segments > 0 ? compare_scratch_bytes(segments) : 0; }

hbp_status hbp_compare(int32_t dtype, int32_t segments, int64_t elems, const void* a, const void* b, double* out,
                       void* scratch, size_t scratch_bytes, void* cuda_stream) {
  if (dtype != HBP_F32 && dtype != HBP_BF16) return HBP_ERR_DTYPE;
  if (segments <= 0 || segments > 65535 || elems <= 0) return HBP_ERR_SHAPE;
  if (!a || !b || !out || !scratch) return HBP_ERR_INVALID_ARG;
  if (((uintptr_t)out | (uintptr_t)scratch) & 7u) return HBP_ERR_SHAPE;
  if (scratch_bytes < compare_scratch_bytes(segments)) return HBP_ERR_WORKSPACE;
  Launcher lc;
  lc.stream = (cudaStream_t)cuda_stream;
  compare_segments(lc, dtype, a, b, segments, elems, out, (double*)scratch);
  return lc.err == cudaSuccess ? HBP_OK : HBP_ERR_CUDA;
}

hbp_status hbp_cumsumprod_scratch_bytes(int32_t dtype, int32_t L, int64_t rows, int32_t d, size_t* bytes) {
  if (!bytes) return HBP_ERR_INVALID_ARG;
  if (dtype != HBP_F32 && dtype != HBP_BF16) return HBP_ERR_DTYPE;
  if (L <= 0 || rows <= 0 || d <= 0 || d % (dtype == HBP_F32 ? 4 : 8)) return HBP_ERR_SHAPE;
  *bytes = scan_scratch_bytes(dtype, L, rows, d);
  return HBP_OK;
}

hbp_status hbp_cumsumprod(int32_t dtype, int32_t gate, int32_t loss, int32_t L, int64_t rows, int32_t d, const void* u,
                          const void* delta, const void* a, void* g, void* scratch, size_t scratch_bytes,
                          void* cuda_stream) {
  return hbp_cumsumprod_status(dtype, gate, loss, L, rows, d, u, delta, a, g, scratch, scratch_bytes, nullptr, cuda_stream);
}

hbp_status hbp_cumsumprod_status(int32_t dtype, int32_t gate, int32_t loss, int32_t L, int64_t rows, int32_t d,
                                 const void* u, const void* delta, const void* a, void* g, void* scratch,
                                 size_t scratch_bytes, int32_t* status, void* cuda_stream) {
  size_t need = 0;
  if ((uintptr_t)status & 3u) return HBP_ERR_SHAPE;
  hbp_status st = hbp_cumsumprod_scratch_bytes(dtype, L, rows, d, &need);
  if (st != HBP_OK) return st;
  if (!delta || !g) return HBP_ERR_INVALID_ARG;
  if (gate < 0 || gate > HBP_GATE_CHANNEL_PER_STEP || (loss != HBP_LOSS_FINAL && loss != HBP_LOSS_EVERY_STEP))
    return HBP_ERR_UNSUPPORTED;
  if (gate != HBP_GATE_ONE && !a) return HBP_ERR_INVALID_ARG;
  if (misaligned(u) || misaligned(delta) || misaligned(a) || misaligned(g) || misaligned(scratch)) return HBP_ERR_SHAPE;
  if (need > 0 && (!scratch || scratch_bytes < need)) return HBP_ERR_WORKSPACE;
  Launcher lc;
  lc.stream = (cudaStream_t)cuda_stream;
  const int64_t state = rows * d;
  const size_t es = dtype == HBP_F32 ? 4 : 2;
  const char* dl = loss == HBP_LOSS_EVERY_STEP ? (const char*)delta + (size_t)L * state * es : (const char*)delta;
  copy_state(lc, dtype, (char*)g + (size_t)L * state * es, dl, state);
  ScanArgs s;
  s.dtype = dtype; s.L = L; s.l_lo = 0; s.l_hi = L; s.rows = rows; s.d = d;
  s.u = u; s.delta = delta; s.loss = loss; s.a = a; s.gate = gate; s.g = g;
  s.scratch = scratch; s.scratch_bytes = scratch_bytes;
  s.status = status;
  scan_reverse(lc, s);
  return lc.err == cudaSuccess ? HBP_OK : HBP_ERR_CUDA;
}

}  // extern "C"
