// C ABI of libhbp: configuration checks, workspace carve-up and the kernel sequences of
// hbp_forward / hbp_backward / hbp_exact.  No device memory is allocated here; every buffer is either
// the caller's or a slice of the caller's workspace.
#include <cstdlib>
#include <cstring>
#include <new>

#include "hbp_internal.h"

namespace hbp {
bool g_force_simt = false;

void gemm(Launcher& lc, const GemmArgs& g, int* status_word) {
  if (!g_force_simt && g.in_dtype == HBP_BF16 && gemm_tc(lc, g, status_word)) return;
  gemm_simt(lc, g);
}
}  // namespace hbp

using namespace hbp;

struct hbp_ctx {
  hbp_config cfg;
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
  char* Z = nullptr;       // [layers][N][h] MLP pre-activations
  float* xres = nullptr;   // [N][d] float master of the residual stream (bf16 only)
  char* U = nullptr;       // [steps][N][d] block VJP outputs (dY before the LayerNorm finish)
  char* H1 = nullptr;      // [group][N][h] dZ
  char* H2 = nullptr;      // [group][N][h] gelu(Z)
  char* C = nullptr;       // RNN: [T][B][d] tanh outputs
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
};

namespace {

constexpr size_t kAlign = 256;
constexpr int kGateBlocks = 256;
constexpr int kMaxSplit = 64;

inline size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

hbp_status check_config(const hbp_config* c) {
  if (!c) return HBP_ERR_INVALID_ARG;
  if (c->dtype != HBP_F32 && c->dtype != HBP_BF16) return HBP_ERR_DTYPE;
  if (c->block < 0 || c->block > HBP_BLOCK_PRELN_TRANSFORMER) return HBP_ERR_UNSUPPORTED;
  if (c->gate < 0 || c->gate > HBP_GATE_CHANNEL_PER_STEP) return HBP_ERR_UNSUPPORTED;
  if (c->loss != HBP_LOSS_FINAL && c->loss != HBP_LOSS_EVERY_STEP) return HBP_ERR_UNSUPPORTED;
  const int v = c->dtype == HBP_F32 ? 4 : 8;
  if (c->L <= 0 || c->d <= 0 || c->tokens <= 0) return HBP_ERR_SHAPE;
  if (c->d % v) return HBP_ERR_SHAPE;
  if (c->d / v > 1024) return HBP_ERR_SHAPE;  // one block per row in the LayerNorm kernels
  if (c->block == HBP_BLOCK_RNN_TANH) {
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
  if (f.dtype == HBP_BF16 && f.block != HBP_BLOCK_RNN_TANH) c->xres = (float*)take(N * d * 4);
  c->partial_floats = (size_t)kGateBlocks * d;
  if (f.block == HBP_BLOCK_RNN_TANH) {
    c->C = take(steps * N * d * es);
    c->scan_scratch_bytes = scan_scratch_bytes(f.dtype, f.L, f.tokens, f.d);
    c->scan_scratch = take(c->scan_scratch_bytes);
    const size_t wmax = d * (d > (size_t)f.in_dim ? d : (size_t)f.in_dim);
    if ((size_t)kMaxSplit * wmax > c->partial_floats) c->partial_floats = (size_t)kMaxSplit * wmax;
  } else {
    if (c->preln) {
      c->Y = take(steps * N * d * es);
      c->rstd = (float*)take(steps * N * 4);
    }
    c->Z = take((size_t)c->layers * N * h * es);
    const size_t per_layer = N * h * es;
    size_t grp = ((size_t)6 << 30) / per_layer;
    if (grp < 1) grp = 1;
    if (grp > (size_t)c->layers) grp = (size_t)c->layers;
    c->group = (int)grp;
    c->H1 = take(grp * per_layer);
    c->H2 = take(grp * per_layer);
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
  int64_t gate_stride(int step_stride) const {
    return c->cfg.gate == HBP_GATE_CHANNEL_PER_STEP ? (int64_t)step_stride * d : 0;
  }
  GemmArgs base_args() const {
    GemmArgs a;
    a.in_dtype = c->cfg.dtype;
    return a;
  }
  void run_gemm(const GemmArgs& a) { gemm(lc, a, c->status); }
  hbp_status result() const { return lc.err == cudaSuccess ? HBP_OK : HBP_ERR_CUDA; }

  // state/step index of MLP layer b and of attention layer b
  int mlp_step(int b) const { return c->cfg.block == HBP_BLOCK_PRELN_TRANSFORMER ? 2 * b + 1 : b; }
  int step_stride() const { return c->cfg.block == HBP_BLOCK_PRELN_TRANSFORMER ? 2 : 1; }
  // operand of W1 for layer b: LayerNorm output or the raw state
  const char* mlp_operand(int b) const {
    return c->preln ? at(c->Y, (int64_t)mlp_step(b) * state) : at(x_all, (int64_t)mlp_step(b) * state);
  }

  // ---- MLP block: u = J^T g for layers [b0, b1) (b1 - b0 <= group), from states g[step+1] -------
  // dA = G W2, dZ = dA * gelu'(Z) -> H1;  dY = dZ W1 -> U[step].  want_act also writes gelu(Z) -> H2.
  void mlp_vjp(int b0, int b1, bool want_act, bool want_dy) {
    const int nb = b1 - b0, ss = step_stride();
    GemmArgs a = base_args();
    a.M = (int)N; a.N = (int)h; a.K = (int)d; a.batch = nb;
    a.A = at(g, (int64_t)(mlp_step(b0) + 1) * state); a.a_sm = d; a.a_sk = 1; a.a_sb = ss * state;
    a.B = at(p->W2, (int64_t)b0 * d * h); a.b_sn = 1; a.b_sk = h; a.b_sb = d * h;
    a.epi = EPI_DGELU;
    a.E = at(c->Z, (int64_t)b0 * N * h); a.lde = h; a.e_sb = N * h;
    a.D = c->H1; a.ldd = h; a.d_sb = N * h;
    if (want_act) { a.D2 = c->H2; a.ldd2 = h; a.d2_sb = N * h; }
    run_gemm(a);
    if (!want_dy) return;
    GemmArgs b = base_args();
    b.M = (int)N; b.N = (int)d; b.K = (int)h; b.batch = nb;
    b.A = c->H1; b.a_sm = h; b.a_sk = 1; b.a_sb = N * h;
    b.B = at(p->W1, (int64_t)b0 * h * d); b.b_sn = 1; b.b_sk = d; b.b_sb = h * d;
    b.epi = EPI_STORE;
    b.D = at(c->U, (int64_t)mlp_step(b0) * state); b.ldd = d; b.d_sb = ss * state;
    run_gemm(b);
  }
  // dW2 = G^T gelu(Z), dW1 = dZ^T y for layers [b0, b1); needs H1, H2 from mlp_vjp(want_act).
  void mlp_wgrad(int b0, int b1, const hbp_grads* gr) {
    const int nb = b1 - b0, ss = step_stride();
    GemmArgs a = base_args();
    a.M = (int)d; a.N = (int)h; a.K = (int)N; a.batch = nb;
    a.A = at(g, (int64_t)(mlp_step(b0) + 1) * state); a.a_sm = 1; a.a_sk = d; a.a_sb = ss * state;
    a.B = c->H2; a.b_sn = 1; a.b_sk = h; a.b_sb = N * h;
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
    run_gemm(a);
    AttnArgs t;
    t.dtype = f.dtype; t.batch = nb * f.batch; t.seq = f.seq; t.heads = f.n_heads; t.head_dim = f.head_dim;
    t.qkv = at(c->QKV, (int64_t)b0 * 3 * state);
    t.o = at(c->O, (int64_t)b0 * state);
    t.lse = c->lse + (int64_t)b0 * f.batch * f.n_heads * f.seq;
    t.d_o = at(c->dO, (int64_t)b0 * state);
    t.d_qkv = at(c->dQKV, (int64_t)b0 * 3 * state);
    t.delta_rows = c->drow + (int64_t)b0 * f.batch * f.n_heads * f.seq;
    attention_bwd(lc, t);
    if (!want_dy) return;
    GemmArgs b = base_args();  // dY = [dQ dK dV] [Wq; Wk; Wv]
    b.M = (int)N; b.N = (int)d; b.K = (int)(3 * d); b.batch = nb;
    b.A = at(c->dQKV, (int64_t)b0 * 3 * state); b.a_sm = 3 * d; b.a_sk = 1; b.a_sb = 3 * state;
    b.B = at(c->Wqkv, (int64_t)b0 * 3 * d * d); b.b_sn = 1; b.b_sk = d; b.b_sb = 3 * d * d;
    b.epi = EPI_STORE;
    b.D = at(c->U, (int64_t)(2 * b0) * state); b.ldd = d; b.d_sb = 2 * state;
    run_gemm(b);
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
  // u_t = (g_{t+1} * (1 - c_t^2)) W for every t at once (one GEMM over T*B rows)
  void rnn_vjp_all() {
    const int T = c->cfg.L;
    GemmArgs a = base_args();
    a.M = (int)(T * N); a.N = (int)d; a.K = (int)d;
    a.A = at(g, state); a.A2 = c->C; a.a_sm = d; a.a_sk = 1;
    a.B = p->W; a.b_sn = 1; a.b_sk = d;
    a.epi = EPI_STORE; a.D = c->U; a.ldd = d;
    run_gemm(a);
  }
  void rnn_wgrad(const hbp_grads* gr) {
    const int T = c->cfg.L;
    const int64_t rows = (int64_t)T * N, in = c->cfg.in_dim;
    int split = (int)(rows / 2048);
    if (split < 1) split = 1;
    if (split > kMaxSplit) split = kMaxSplit;
    for (int w = 0; w < 2; ++w) {
      GemmArgs a = base_args();  // dW = dZ^T H (H = states 0..T-1), dU = dZ^T X
      a.M = (int)d; a.N = w == 0 ? (int)d : (int)in; a.K = (int)rows;
      a.A = at(g, state); a.A2 = c->C; a.a_sm = 1; a.a_sk = d;
      a.B = w == 0 ? x_all : inputs; a.b_sn = 1; a.b_sk = a.N;
      a.epi = EPI_STORE; a.d_f32 = true;
      a.D = w == 0 ? gr->dW : gr->dU; a.ldd = a.N;
      if (split > 1) { a.splitk = split; a.partial = c->partial; }
      if (a.D) run_gemm(a);
    }
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

  ScanArgs scan_args(int lo, int hi, bool with_u) const {
    ScanArgs s;
    s.dtype = c->cfg.dtype; s.L = c->steps; s.l_lo = lo; s.l_hi = hi; s.rows = N; s.d = (int)d;
    s.u = with_u ? c->U : nullptr;
    s.delta = delta; s.loss = c->cfg.loss;
    s.a = p->a; s.gate = c->cfg.gate;
    s.g = g;
    if (with_u && c->preln) { s.xhat = c->Y; s.rstd = c->rstd; }
    s.scratch = c->scan_scratch; s.scratch_bytes = c->scan_scratch_bytes;
    return s;
  }
  void set_last_state() {
    const char* dl = c->cfg.loss == HBP_LOSS_EVERY_STEP ? at(delta, (int64_t)c->steps * state) : delta;
    copy_state(lc, c->cfg.dtype, at(g, (int64_t)c->steps * state), dl, state);
  }
};

hbp_status check_call(hbp_ctx* ctx, const hbp_params* p, bool need_forward) {
  if (!ctx || !p) return HBP_ERR_INVALID_ARG;
  if (need_forward && !ctx->forward_done) return HBP_ERR_STATE;
  const hbp_config& f = ctx->cfg;
  if (f.block == HBP_BLOCK_RNN_TANH) {
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
  if (f.block == HBP_BLOCK_RNN_TANH) return (g->dW && g->dU) ? HBP_OK : HBP_ERR_INVALID_ARG;
  if (!g->dW1 || !g->dW2) return HBP_ERR_INVALID_ARG;
  if (f.block == HBP_BLOCK_PRELN_TRANSFORMER && (!g->dWq || !g->dWk || !g->dWv || !g->dWo)) return HBP_ERR_INVALID_ARG;
  return HBP_OK;
}

bool misaligned(const void* p) { return ((uintptr_t)p & 15u) != 0; }

}  // namespace
