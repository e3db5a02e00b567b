// Split-model runtime and C ABI: context, workspace plan, the per-step kernel schedules of
// Algorithm 1 (client forward, server step, client backward, aggregation) and the stand-alone
// operator entry points.  Host code only; every device operation is a launcher from kernels.h.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <string>
#include <vector>

#include "../../include/splitlora.h"
#include "kernels.h"

using namespace sl;

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct FrozenLayer {
  const void *ln1g = nullptr, *ln1b = nullptr, *qkvw = nullptr, *qkvb = nullptr, *projw = nullptr,
             *projb = nullptr, *ln2g = nullptr, *ln2b = nullptr, *fc1w = nullptr, *fc1b = nullptr,
             *fc2w = nullptr, *fc2b = nullptr;
  void *qkvwT = nullptr, *projwT = nullptr, *fc1wT = nullptr, *fc2wT = nullptr;   // [in, out] copies
};

// What one block keeps from its forward pass for its backward pass.
struct LayerBuf {
  void *u = nullptr, *hcat = nullptr, *qkv = nullptr, *o = nullptr, *x_mid = nullptr, *z = nullptr,
       *x_out = nullptr;
  float *mean1 = nullptr, *rstd1 = nullptr, *mean2 = nullptr, *rstd2 = nullptr, *lse = nullptr;
  const void* x_in = nullptr;     // base (row 0) of the buffer the block read its input from
  void* hcat_o = nullptr;         // down-projected input of an adapter on the attention output projection
  // Adapter compute copies of this layer: `cl` holds one set per client, stacked (blocks the clients
  // run), `sv` the server's single set (blocks the server runs).  A block between the shallowest and the
  // deepest client cut is run by both sides and has both.
  struct Copies {
    void *Acat = nullptr, *AcatT = nullptr, *Bext = nullptr, *BextT = nullptr;
    void *AcatO = nullptr, *AcatOT = nullptr, *BextO = nullptr, *BextOT = nullptr;   // output projection
  } cl, sv;
};

// The rows one call of a block works on: `rows` consecutive token rows from row0, which belong to the
// clients client0, client0 + 1, ... (client side: each with its own adapters) or to the server's batch.
struct Span {
  int row0 = 0, rows = 0, client0 = 0, n_clients = 0;
  bool client = false;
};

struct ProfRec { int cls; cudaEvent_t a, b; };

// Arena cursor: with base == nullptr it only measures.
struct Arena {
  char* base; size_t off = 0;
  explicit Arena(char* b) : base(b) {}
  void* take(size_t bytes) {
    off = align_up(off, 256);
    void* p = base ? base + off : nullptr;
    off += bytes;
    return p;
  }
};

}  // namespace

struct splitlora_ctx {
  splitlora_config cfg;
  cudaStream_t st = nullptr;
  std::string err;
  int dt = 0; size_t es = 4;
  int M = 0, nseq = 0, d = 0, F = 0, V = 0, Vpad = 0, L = 0, cut = 0, K = 0, rows_per_client = 0;
  int cmin = 0;               // first block with server adapters (= cut unless clients are cut at different depths)
  std::vector<int> client_cut;   // per-client cut, non-decreasing (empty: every client is cut at `cut`)
  int r = 0, rp = 0, ext = 0, ke = 0, n_targets = 0;
  int nq = 0;                 // adapted slices of the fused qkv projection (targets 0..nq-1)
  bool has_o = false;         // adapter on the attention output projection (target index nq)
  int ext_o = 0;
  bool llama = false;
  int Fz = 0;                 // width of the saved MLP pre-activation: d_ff, or 2*d_ff (gate | up)
  int slice_idx[4] = {0, 0, 0, 0};
  uint32_t target_bit[4] = {0, 0, 0, 0};
  float scale = 1.f;
  bool tc = false;
  // frozen
  const void *wte = nullptr, *wpe = nullptr, *lnfg = nullptr, *lnfb = nullptr, *headw = nullptr;
  void* wteT = nullptr;       // transposed head [d, Vpad]
  float* rope_table = nullptr;
  std::vector<float> rope_host;
  std::vector<FrozenLayer> fl;
  int n_bound = 0;
  // workspace
  char* ws = nullptr; size_t ws_bytes = 0;
  std::vector<LayerBuf> lb;
  int64_t per_layer = 0, Pc = 0, Ps = 0;     // floats per layer, per client set, server set
  float *cp = nullptr, *cg = nullptr, *cm = nullptr, *cv = nullptr;   // client params/grads/moments [K, Pc]
  float *sp = nullptr, *sg = nullptr, *sm = nullptr, *sv = nullptr;   // server [Ps]
  float* agg_sum = nullptr;   // [Pc]: weighted sum of the local clients' adapters (clients spread over devices)
  void *emb = nullptr, *u2 = nullptr, *act = nullptr, *xf = nullptr, *logits = nullptr;
  float *meanf = nullptr, *rstdf = nullptr, *row_loss = nullptr, *rowdot = nullptr, *loss_dev = nullptr,
        *grad_scratch = nullptr;
  size_t grad_scratch_floats = 0;
  int *n_valid = nullptr, *status = nullptr;
  void *g_a = nullptr, *g_b = nullptr, *g_dz = nullptr, *g_du2 = nullptr, *g_dxmid = nullptr, *g_do = nullptr,
       *g_dqkv = nullptr, *g_dhcat = nullptr, *g_du = nullptr, *g_dhcat_o = nullptr;
  void *S = nullptr, *dS = nullptr;
  int32_t *tok_dev = nullptr, *lab_dev = nullptr;
  // state
  bool client_copies_dirty = true, server_copies_dirty = true;
  bool have_client_fwd = false;
  // sharding over devices: global loss normaliser (0: local count) and server update left to the caller
  int64_t loss_normalizer = 0;
  bool defer_server_update = false;
  std::vector<int> client_rank;             // per-client adapter rank (empty: every client has lora_r)
  int64_t round_index = 0, server_steps = 0, client_steps = 0;
  int64_t launches = 0;
  // profiling
  int prof_on = 0;            // 0 off, 1 every launch class, 2 the tensor-bound linear classes only
  std::vector<std::string> prof_names;
  std::map<std::string, int> prof_ids;
  std::vector<ProfRec> prof_recs;
  std::vector<cudaEvent_t> event_pool;
};

namespace {

int fail(splitlora_ctx* c, int code, const std::string& msg) {
  if (c) c->err = msg;
  return code;
}

#define CK(ctx, expr)                                                                         \
  do {                                                                                        \
    cudaError_t e__ = (expr);                                                                 \
    if (e__ != cudaSuccess)                                                                   \
      return fail(ctx, SPLITLORA_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__)); \
  } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int validate(const splitlora_config* c, std::string* why) {
  auto bad = [&](const char* m) { *why = m; return SPLITLORA_ERR_ARG; };
  if (!c) return bad("null config");
  // cut == n_layer puts every block on the clients (the server keeps the final norm and the head):
  // the federated-LoRA baseline of Sec. IV as a degenerate case of the same round
  if (c->n_layer < 1 || c->cut < 1 || c->cut > c->n_layer) return bad("need 1 <= cut <= n_layer");
  if (c->cut_min < 0 || c->cut_min > c->cut) return bad("need 0 <= cut_min <= cut");
  if (c->d_model < 8 || c->n_head < 1 || c->d_model % c->n_head != 0) return bad("d_model must be a multiple of n_head");
  if (c->d_model % 8 != 0 || c->d_ff % 8 != 0) return bad("d_model and d_ff must be multiples of 8");
  if (c->d_model / c->n_head > 128) return bad("head width above 128");
  if (c->vocab < 2 || c->max_seq < 1 || c->seq < 1 || c->seq > c->max_seq) return bad("bad vocab / seq");
  if (c->lora_r < 1 || c->lora_r > 64) return bad("lora_r must be in 1..64");
  if ((c->lora_targets & 7u) == 0 || (c->lora_targets & ~15u))
    return bad("lora_targets must name at least one of q, k, v, and optionally o");
  if (c->arch != SPLITLORA_ARCH_GPT && c->arch != SPLITLORA_ARCH_LLAMA) return bad("bad arch");
  if (c->arch == SPLITLORA_ARCH_LLAMA) {
    const int dh = c->d_model / c->n_head, vec = c->dtype == SPLITLORA_DTYPE_BF16 ? 8 : 4;
    if (dh % 2 != 0 || (dh / 2) % vec != 0) return bad("half the head width must be a multiple of the 16-byte vector width");
    if (!(c->rope_theta > 0.f)) return bad("rope_theta must be positive");
  }
  if (c->n_clients < 1 || c->n_clients > AGG_MAX_CLIENTS) return bad("n_clients must be in 1..64");
  if (c->batch_per_client < 1) return bad("batch_per_client must be positive");
  if (((int64_t)c->batch_per_client * c->seq) % 256 != 0 && c->n_clients > 1)
    return bad("batch_per_client * seq must be a multiple of 256 (client segments align with kernel tiles)");
  if (c->dtype != SPLITLORA_DTYPE_FP32 && c->dtype != SPLITLORA_DTYPE_BF16) return bad("bad dtype");
  if (c->optimizer != SPLITLORA_OPT_SGD && c->optimizer != SPLITLORA_OPT_ADAMW) return bad("bad optimizer");
  if (c->agg_interval < 1) return bad("agg_interval must be >= 1");
  if (!(c->norm_eps > 0.f)) return bad("norm_eps must be positive");
  return SPLITLORA_OK;
}

void derive(splitlora_ctx* c) {
  const splitlora_config& g = c->cfg;
  c->dt = g.dtype; c->es = dtype_size(g.dtype);
  c->L = g.n_layer; c->cut = g.cut; c->K = g.n_clients;
  c->d = g.d_model; c->F = g.d_ff; c->V = g.vocab;
  c->Vpad = (int)align_up((size_t)g.vocab, 64);
  c->nseq = g.n_clients * g.batch_per_client;
  c->rows_per_client = g.batch_per_client * g.seq;
  c->M = c->nseq * g.seq;
  c->r = g.lora_r; c->rp = (int)align_up((size_t)g.lora_r, 16);
  c->n_targets = 0;
  for (int s = 0; s < 3; ++s)
    if (g.lora_targets & (1u << s)) { c->slice_idx[c->n_targets] = s; c->target_bit[c->n_targets] = 1u << s; c->n_targets++; }
  c->nq = c->n_targets;
  c->has_o = (g.lora_targets & SPLITLORA_TARGET_O) != 0;
  if (c->has_o) { c->slice_idx[c->n_targets] = 0; c->target_bit[c->n_targets] = SPLITLORA_TARGET_O; c->n_targets++; }
  c->ke = c->nq * c->rp;
  c->ext = (int)align_up((size_t)c->ke, EXT_BLOCK);
  c->ext_o = c->has_o ? (int)align_up((size_t)c->rp, EXT_BLOCK) : 0;
  c->llama = g.arch == SPLITLORA_ARCH_LLAMA;
  c->Fz = c->llama ? 2 * g.d_ff : g.d_ff;
  c->scale = g.lora_alpha / (float)g.lora_r;
  c->per_layer = (int64_t)c->n_targets * 2 * c->r * c->d;
  c->cmin = g.cut_min > 0 ? g.cut_min : g.cut;
  c->Pc = c->per_layer * c->cut;
  c->Ps = c->per_layer * (c->L - c->cmin);
  c->tc = (g.dtype == SPLITLORA_DTYPE_BF16) && g.use_tensor_cores != 0;
}

// Lays out the workspace.  With ws == nullptr only the size is computed.
size_t plan(splitlora_ctx* c, char* ws) {
  Arena a(ws);
  const size_t es = c->es;
  const size_t M = c->M, d = c->d, F = c->F, ext = c->ext, Fz = c->Fz, ext_o = c->ext_o;
  c->status = (int*)a.take(256);
  c->loss_dev = (float*)a.take(256);
  c->n_valid = (int*)a.take(256);
  if (c->llama) c->rope_table = (float*)a.take((size_t)c->cfg.seq * (d / c->cfg.n_head / 2) * 8);
  // adapters: masters, gradients, moments
  c->cp = (float*)a.take((size_t)c->K * c->Pc * 4); c->cg = (float*)a.take((size_t)c->K * c->Pc * 4);
  c->cm = (float*)a.take((size_t)c->K * c->Pc * 4); c->cv = (float*)a.take((size_t)c->K * c->Pc * 4);
  c->sp = (float*)a.take((size_t)c->Ps * 4); c->sg = (float*)a.take((size_t)c->Ps * 4);
  c->sm = (float*)a.take((size_t)c->Ps * 4); c->sv = (float*)a.take((size_t)c->Ps * 4);
  c->agg_sum = (float*)a.take((size_t)c->Pc * 4);
  c->fl.resize(c->L);
  c->lb.resize(c->L);
  for (int l = 0; l < c->L; ++l) {
    FrozenLayer& f = c->fl[l];
    f.qkvwT = a.take(3 * d * d * es); f.projwT = a.take(d * d * es);
    f.fc1wT = a.take(Fz * d * es); f.fc2wT = a.take(d * F * es);
    LayerBuf& b = c->lb[l];
    for (int side = 0; side < 2; ++side) {
      if (side == 0 ? l >= c->cut : l < c->cmin) continue;
      const size_t G = side == 0 ? c->K : 1;
      LayerBuf::Copies& k = side == 0 ? b.cl : b.sv;
      k.Acat = a.take(G * ext * d * es); k.AcatT = a.take(G * d * ext * es);
      k.Bext = a.take(G * 3 * d * ext * es); k.BextT = a.take(G * ext * 3 * d * es);
      if (c->has_o) {
        k.AcatO = a.take(G * ext_o * d * es); k.AcatOT = a.take(G * d * ext_o * es);
        k.BextO = a.take(G * d * ext_o * es); k.BextOT = a.take(G * ext_o * d * es);
      }
    }
    if (c->has_o) b.hcat_o = a.take(M * ext_o * es);
    b.u = a.take(M * d * es); b.hcat = a.take(M * ext * es); b.qkv = a.take(M * 3 * d * es);
    b.o = a.take(M * d * es); b.x_mid = a.take(M * d * es); b.z = a.take(M * Fz * es);
    b.x_out = a.take(M * d * es);
    b.mean1 = (float*)a.take(M * 4); b.rstd1 = (float*)a.take(M * 4);
    b.mean2 = (float*)a.take(M * 4); b.rstd2 = (float*)a.take(M * 4);
    b.lse = (float*)a.take((size_t)c->nseq * c->cfg.n_head * c->cfg.seq * 4);
  }
  c->wteT = a.take(d * (size_t)c->Vpad * es);
  c->emb = a.take(M * d * es); c->u2 = a.take(M * d * es); c->act = a.take(M * F * es);
  c->xf = a.take(M * d * es); c->logits = a.take(M * (size_t)c->Vpad * es);
  c->meanf = (float*)a.take(M * 4); c->rstdf = (float*)a.take(M * 4); c->row_loss = (float*)a.take(M * 4);
  c->rowdot = (float*)a.take((size_t)c->nseq * c->cfg.n_head * c->cfg.seq * 4);
  c->grad_scratch_floats = lora_grad_scratch_floats(c->M, c->nq * c->r, c->d);
  c->grad_scratch = (float*)a.take(c->grad_scratch_floats * 4);
  if (c->has_o) c->g_dhcat_o = a.take(M * ext_o * es);
  c->g_a = a.take(M * d * es); c->g_b = a.take(M * d * es); c->g_dz = a.take(M * Fz * es);
  c->g_du2 = a.take(M * d * es); c->g_dxmid = a.take(M * d * es); c->g_do = a.take(M * d * es);
  c->g_dqkv = a.take(M * 3 * d * es); c->g_dhcat = a.take(M * ext * es); c->g_du = a.take(M * d * es);
  c->S = a.take(M * d * es); c->dS = a.take(M * d * es);
  c->tok_dev = (int32_t*)a.take(M * 4); c->lab_dev = (int32_t*)a.take(M * 4);
  return align_up(a.off, 256);
}

// ---- profiling -----------------------------------------------------------------------------
struct Scope {
  splitlora_ctx* c; int cls = -1; cudaEvent_t a = nullptr, b = nullptr;
  Scope(splitlora_ctx* ctx, const char* name, int kernels) : c(ctx) {
    c->launches += kernels;
    if (!c->prof_on) return;
    if (c->prof_on == 2 && !std::strstr(name, "linear_") && std::strncmp(name, "head_", 5) != 0) return;
    auto it = c->prof_ids.find(name);
    if (it == c->prof_ids.end()) {
      cls = (int)c->prof_names.size();
      c->prof_names.push_back(name); c->prof_ids[name] = cls;
    } else cls = it->second;
    auto get = [&]() {
      cudaEvent_t e;
      if (!c->event_pool.empty()) { e = c->event_pool.back(); c->event_pool.pop_back(); }
      else cudaEventCreate(&e);
      return e;
    };
    a = get(); b = get();
    cudaEventRecord(a, c->st);
  }
  ~Scope() {
    if (cls < 0) return;
    cudaEventRecord(b, c->st);
    c->prof_recs.push_back({cls, a, b});
  }
};

cudaError_t linear(splitlora_ctx* c, const char* name, const GemmArgs& a) {
  Scope s(c, name, 1);
  if (c->tc && gemm_tc_supported(a)) return gemm_tc(a, c->status, c->st);
  return gemm_simt(a, c->st);
}

GemmArgs base_args(splitlora_ctx* c, const void* X, int64_t ldx, const void* W, int64_t ldw, void* Y, int64_t ldy,
                   int M, int N, int K) {
  GemmArgs a;
  a.dtype = c->dt; a.X = X; a.ldx = ldx; a.W = W; a.ldw = ldw; a.Y = Y; a.ldy = ldy; a.M = M; a.N = N; a.K = K;
  a.gelu_tanh = c->cfg.gelu_tanh;
  return a;
}

bool all_frozen_bound(const splitlora_ctx* c) { return c->n_bound == (c->llama ? 3 + 6 * c->L : 4 + 12 * c->L); }

cudaError_t refresh_side(splitlora_ctx* c, bool client) {
  AdapterCopyArgs a;
  a.dtype = c->dt;
  a.a_gs = a.b_gs = client ? c->Pc : 0;
  a.a_ts = a.b_ts = (int64_t)2 * c->r * c->d;
  a.r = c->r; a.rp = c->rp; a.d_in = c->d; a.d_out = c->d;
  a.scale = c->scale;
  a.G = client ? c->K : 1;
  const int l0 = client ? 0 : c->cmin, l1 = client ? c->cut : c->L;
  for (int l = l0; l < l1; ++l) {
    const float* base = (client ? c->cp : c->sp) + (size_t)(l - l0) * c->per_layer;
    const LayerBuf::Copies& k = client ? c->lb[l].cl : c->lb[l].sv;
    {  // the adapted slices of the fused qkv projection
      a.A = base; a.B = a.A + (size_t)c->r * c->d;
      a.n_targets = c->nq; a.n_out = 3 * c->d; a.ext = c->ext;
      for (int t = 0; t < 4; ++t) a.slice_off[t] = c->slice_idx[t] * c->d;
      a.Acat = k.Acat; a.AcatT = k.AcatT; a.Bext = k.Bext; a.BextT = k.BextT;
      Scope s(c, "adapter_copies", 1);
      cudaError_t e = refresh_adapter_copies(a, c->st);
      if (e != cudaSuccess) return e;
    }
    if (c->has_o) {  // the output projection: a LoRA layer of its own
      a.A = base + (size_t)c->nq * 2 * c->r * c->d; a.B = a.A + (size_t)c->r * c->d;
      a.n_targets = 1; a.n_out = c->d; a.ext = c->ext_o;
      for (int t = 0; t < 4; ++t) a.slice_off[t] = 0;
      a.Acat = k.AcatO; a.AcatT = k.AcatOT; a.Bext = k.BextO; a.BextT = k.BextOT;
      Scope s(c, "adapter_copies", 1);
      cudaError_t e = refresh_adapter_copies(a, c->st);
      if (e != cudaSuccess) return e;
    }
  }
  return cudaSuccess;
}

// LayerNorm or RMSNorm over M rows, by architecture (mean is unused by RMSNorm)
cudaError_t norm_forward(splitlora_ctx* c, int M, const void* x, const void* g, const void* b, void* y, float* mean,
                         float* rstd) {
  Scope s(c, "layernorm_fwd", 1);
  if (c->llama) return rmsnorm_fwd(c->dt, x, g, y, rstd, M, c->d, c->cfg.norm_eps, c->st);
  return layernorm_fwd(c->dt, x, g, b, y, mean, rstd, M, c->d, c->cfg.norm_eps, c->st);
}
cudaError_t norm_backward(splitlora_ctx* c, int M, const void* dy, const void* x, const void* g, const float* mean,
                          const float* rstd, const void* resid, void* dx) {
  Scope s(c, "layernorm_bwd", 1);
  if (c->llama) return rmsnorm_bwd(c->dt, dy, x, g, rstd, resid, dx, M, c->d, c->st);
  return layernorm_bwd(c->dt, dy, x, g, mean, rstd, resid, dx, M, c->d, c->st);
}

// Spans of a block.  Clients are ordered by non-decreasing cut, so the clients that run block l
// themselves are a suffix {i : cut_i > l} and the server's batch at block l is the prefix {i : cut_i <= l}.
int cut_of(const splitlora_ctx* c, int i) { return c->client_cut.empty() ? c->cut : c->client_cut[i]; }
bool uniform_cut(const splitlora_ctx* c) { return c->client_cut.empty(); }
int first_client_above(const splitlora_ctx* c, int l) {       // first client with cut > l (K if none)
  int i = 0;
  while (i < c->K && cut_of(c, i) <= l) ++i;
  return i;
}
Span client_span(const splitlora_ctx* c, int l) {
  Span sp;
  sp.client = true; sp.client0 = first_client_above(c, l); sp.n_clients = c->K - sp.client0;
  sp.row0 = sp.client0 * c->rows_per_client; sp.rows = sp.n_clients * c->rows_per_client;
  return sp;
}
Span server_span(const splitlora_ctx* c, int l) {
  Span sp;
  sp.client = false; sp.client0 = 0; sp.n_clients = first_client_above(c, l);
  sp.row0 = 0; sp.rows = sp.n_clients * c->rows_per_client;
  return sp;
}
// rows [client_a, client_b) of src -> the same rows of dst ([M, d] buffers): a hand-off of those clients
cudaError_t copy_client_rows(splitlora_ctx* c, const void* src, void* dst, int client_a, int client_b) {
  if (client_b <= client_a) return cudaSuccess;
  const size_t off = (size_t)client_a * c->rows_per_client * c->d * c->es;
  const size_t n = (size_t)(client_b - client_a) * c->rows_per_client * c->d * c->es;
  return cudaMemcpyAsync((char*)dst + off, (const char*)src + off, n, cudaMemcpyDeviceToDevice, c->st);
}

// ---- one block -----------------------------------------------------------------------------
// x_in, x_out: bases (row 0) of [M, d] buffers; the block reads and writes the rows of `sp`.
cudaError_t block_forward(splitlora_ctx* c, int l, const Span& sp, const void* x_in, void* x_out) {
  const bool client = sp.client;
  const int M = sp.rows, d = c->d, F = c->F, ext = c->ext, T = c->cfg.seq, H = c->cfg.n_head;
  if (M == 0) return cudaSuccess;
  const int rpg = client ? c->rows_per_client : 0;
  const bool grouped = client && sp.n_clients > 1;
  const size_t es = c->es;
  const FrozenLayer& f = c->fl[l];
  LayerBuf& b = c->lb[l];
  const LayerBuf::Copies& k = client ? b.cl : b.sv;
  auto at = [&](const void* p, size_t ld) { return (void*)((char*)p + (size_t)sp.row0 * ld * es); };        // activations
  auto atf = [&](float* p) { return p + sp.row0; };                                                           // per-row fp32
  auto grp = [&](const void* p, size_t elems) { return (const void*)((const char*)p + (size_t)(client ? sp.client0 : 0) * elems * es); };
  float* lse = b.lse + (size_t)(sp.row0 / T) * H * T;
  b.x_in = x_in;
  const void* xin = at(x_in, d);
  void* u = at(b.u, d); void* hcat = at(b.hcat, ext); void* qkv = at(b.qkv, 3 * d); void* o = at(b.o, d);
  void* x_mid = at(b.x_mid, d); void* z = at(b.z, c->Fz); void* xout = at(x_out, d);
  cudaError_t e;
  if ((e = norm_forward(c, M, xin, f.ln1g, f.ln1b, u, atf(b.mean1), atf(b.rstd1)))) return e;
  {  // h = u A_g^T for every target of the layer, one padded block of `ext` columns
    GemmArgs a = base_args(c, u, d, grp(k.Acat, (size_t)ext * d), d, hcat, ext, M, ext, d);
    a.rows_per_group = rpg; a.w_grouped = grouped;
    if ((e = linear(c, "lora_down_fwd", a))) return e;
  }
  {  // qkv = u Wqkv^T + b + hcat Bext_g^T   (the LoRA linear of Sec. II-C, grouped by client)
    GemmArgs a = base_args(c, u, d, f.qkvw, d, qkv, 3 * d, M, 3 * d, d);
    a.bias = f.qkvb; a.rows_per_group = rpg;
    a.Xe = hcat; a.ldxe = ext; a.We = grp(k.Bext, (size_t)3 * d * ext); a.ldwe = ext; a.Ke = c->ke; a.we_grouped = grouped;
    if ((e = linear(c, "lora_linear_fwd", a))) return e;
  }
  if (c->llama) {
    Scope s(c, "rope", 1);
    if ((e = rope_inplace(c->dt, qkv, c->rope_table, M, T, H, d, 1.0f, c->st))) return e;
  }
  { Scope s(c, "attention_fwd", 1);
    if (c->tc && attention_tc_supported(c->dt, T, H, d))
      e = attention_fwd_tc(qkv, M / T, T, H, d, o, lse, c->status, c->st);
    else
      e = attention_fwd_simt(c->dt, qkv, M / T, T, H, d, o, lse, c->st);
    if (e) return e; }
  void* hcat_o = c->has_o ? at(b.hcat_o, c->ext_o) : nullptr;
  if (c->has_o) {  // h_o = o A_o,g^T
    GemmArgs a = base_args(c, o, d, grp(k.AcatO, (size_t)c->ext_o * d), d, hcat_o, c->ext_o, M, c->ext_o, d);
    a.rows_per_group = rpg; a.w_grouped = grouped;
    if ((e = linear(c, "lora_down_fwd", a))) return e;
  }
  { GemmArgs a = base_args(c, o, d, f.projw, d, x_mid, d, M, d, d);
    a.bias = f.projb; a.epi = EPI_BIAS_RESID; a.R = xin; a.ldr = d;
    if (c->has_o) {
      a.rows_per_group = rpg;
      a.Xe = hcat_o; a.ldxe = c->ext_o; a.We = grp(k.BextO, (size_t)d * c->ext_o); a.ldwe = c->ext_o; a.Ke = c->rp;
      a.we_grouped = grouped;
    }
    if ((e = linear(c, c->has_o ? "lora_linear_fwd" : "linear_fwd", a))) return e; }
  if ((e = norm_forward(c, M, x_mid, f.ln2g, f.ln2b, c->u2, atf(b.mean2), atf(b.rstd2)))) return e;
  if (c->llama) {
    { GemmArgs a = base_args(c, c->u2, d, f.fc1w, d, z, 2 * F, M, 2 * F, d);     // (gate | up)
      if ((e = linear(c, "linear_fwd", a))) return e; }
    { Scope s(c, "swiglu_fwd", 1);
      if ((e = swiglu_fwd(c->dt, z, c->act, M, F, c->st))) return e; }
  } else {
    GemmArgs a = base_args(c, c->u2, d, f.fc1w, d, c->act, F, M, F, d);
    a.bias = f.fc1b; a.epi = EPI_BIAS_GELU; a.Z = z; a.ldz = F;
    if ((e = linear(c, "linear_fwd", a))) return e;
  }
  { GemmArgs a = base_args(c, c->act, F, f.fc2w, F, xout, d, M, d, F);
    a.bias = f.fc2b; a.epi = EPI_BIAS_RESID; a.R = x_mid; a.ldr = d;
    if ((e = linear(c, "linear_fwd", a))) return e; }
  return cudaSuccess;
}

// dy: gradient w.r.t. the block output; dx: gradient w.r.t. the block input, or nullptr when it is not
// needed (first client block: the embedding below it is frozen).  Both are bases of [M, d] buffers; the
// rows of `sp` are read and written.
cudaError_t block_backward(splitlora_ctx* c, int l, const Span& sp, const void* dy_base, void* dx_base) {
  const bool client = sp.client;
  const int M = sp.rows, d = c->d, F = c->F, ext = c->ext, T = c->cfg.seq, H = c->cfg.n_head;
  if (M == 0) return cudaSuccess;
  const int rpg = client ? c->rows_per_client : 0;
  const bool grouped = client && sp.n_clients > 1;
  const size_t es = c->es;
  const FrozenLayer& f = c->fl[l];
  LayerBuf& b = c->lb[l];
  const LayerBuf::Copies& k = client ? b.cl : b.sv;
  auto at = [&](const void* p, size_t ld) { return (void*)((char*)p + (size_t)sp.row0 * ld * es); };
  auto atf = [&](float* p) { return p + sp.row0; };
  auto grp = [&](const void* p, size_t elems) { return (const void*)((const char*)p + (size_t)(client ? sp.client0 : 0) * elems * es); };
  const float* lse = b.lse + (size_t)(sp.row0 / T) * H * T;
  const void* dy = at(dy_base, d);
  void* dx = dx_base ? at(dx_base, d) : nullptr;
  const void* u = at(b.u, d); const void* hcat = at(b.hcat, ext); const void* qkv = at(b.qkv, 3 * d);
  const void* o = at(b.o, d); const void* x_mid = at(b.x_mid, d); const void* z = at(b.z, c->Fz);
  cudaError_t e;
  const int Fz = c->Fz;
  float* gbase = client ? c->cg + (size_t)sp.client0 * c->Pc + (size_t)l * c->per_layer
                        : c->sg + (size_t)(l - c->cmin) * c->per_layer;
  const int64_t gstride = client ? c->Pc : 0;
  if (c->llama) {
    { GemmArgs a = base_args(c, dy, d, f.fc2wT, d, c->act, F, M, F, d);               // d act
      if ((e = linear(c, "linear_bwd", a))) return e; }
    { Scope s(c, "swiglu_bwd", 1);
      if ((e = swiglu_bwd(c->dt, c->act, z, c->g_dz, M, F, c->st))) return e; }
  } else {
    GemmArgs a = base_args(c, dy, d, f.fc2wT, d, c->g_dz, F, M, F, d);
    a.epi = EPI_MUL_GELUGRAD; a.R = z; a.ldr = F;
    if ((e = linear(c, "linear_bwd", a))) return e;
  }
  { GemmArgs a = base_args(c, c->g_dz, Fz, f.fc1wT, Fz, c->g_du2, d, M, d, Fz);
    if ((e = linear(c, "linear_bwd", a))) return e; }
  if ((e = norm_backward(c, M, c->g_du2, x_mid, f.ln2g, atf(b.mean2), atf(b.rstd2), dy, c->g_dxmid))) return e;
  if (c->has_o) {
    // dh_o = (alpha/r) dx_mid B_o,g ;  G_A = dh_o^T o ;  G_B = (alpha/r) dx_mid^T h_o   (Eq. 4-7)
    const void* hcat_o = at(b.hcat_o, c->ext_o);
    { GemmArgs a = base_args(c, c->g_dxmid, d, grp(k.BextOT, (size_t)c->ext_o * d), d, c->g_dhcat_o, c->ext_o, M, c->ext_o, d);
      a.rows_per_group = rpg; a.w_grouped = grouped;
      if ((e = linear(c, "lora_down_bwd", a))) return e; }
    float* gA = gbase + (size_t)c->nq * 2 * c->r * d;
    { Scope s(c, "lora_grad", 2);
      if ((e = lora_grad(c->dt, o, d, 0, d, c->g_dhcat_o, c->ext_o, 0, c->r, c->rp, 1, M, rpg, 1.0f, gA, gstride, 0, d,
                         1, c->grad_scratch, c->st, c->status, c->tc))) return e; }
    { Scope s(c, "lora_grad", 2);
      if ((e = lora_grad(c->dt, c->g_dxmid, d, 0, d, hcat_o, c->ext_o, 0, c->r, c->rp, 1, M, rpg, c->scale,
                         gA + (size_t)c->r * d, gstride, 0, 1, c->r, c->grad_scratch, c->st, c->status, c->tc))) return e; }
  }
  { GemmArgs a = base_args(c, c->g_dxmid, d, f.projwT, d, c->g_do, d, M, d, d);
    if (c->has_o) {
      a.rows_per_group = rpg;
      a.Xe = c->g_dhcat_o; a.ldxe = c->ext_o; a.We = grp(k.AcatOT, (size_t)d * c->ext_o); a.ldwe = c->ext_o; a.Ke = c->rp;
      a.we_grouped = grouped;
    }
    if ((e = linear(c, c->has_o ? "lora_linear_bwd" : "linear_bwd", a))) return e; }
  { Scope s(c, "attention_bwd", c->tc && attention_t5_supported(c->dt, T, H, d) ? 2 : 3);
    if (c->tc && attention_tc_supported(c->dt, T, H, d))
      e = attention_bwd_tc(qkv, o, lse, c->g_do, M / T, T, H, d, c->g_dqkv, c->rowdot, c->status, c->st);
    else
      e = attention_bwd_simt(c->dt, qkv, o, lse, c->g_do, M / T, T, H, d, c->g_dqkv, c->rowdot, c->st);
    if (e) return e; }
  if (c->llama) {  // the gradient of a rotation is the inverse rotation
    Scope s(c, "rope", 1);
    if ((e = rope_inplace(c->dt, c->g_dqkv, c->rope_table, M, T, H, d, -1.0f, c->st))) return e;
  }
  {  // dh = (alpha/r) dqkv B_g for every target (the scale lives in the compute copy)
    GemmArgs a = base_args(c, c->g_dqkv, 3 * d, grp(k.BextT, (size_t)ext * 3 * d), 3 * d, c->g_dhcat, ext, M, ext, 3 * d);
    a.rows_per_group = rpg; a.w_grouped = grouped;
    if (c->tc && c->nq < 3) {
      // only the adapted slices of dqkv contribute (the other rows of the compute copy are zero):
      // contract over those columns alone, which is one third less to read for q and v
      GemmArgs g = a;
      const int lo = c->slice_idx[0], hi = c->slice_idx[c->nq - 1];
      g.X = (const char*)a.X + (size_t)lo * d * c->es;
      g.W = (const char*)a.W + (size_t)lo * d * c->es;
      g.K = c->nq * d;
      if (hi - lo + 1 > c->nq) { g.k_gap_begin = d; g.k_gap_len = d; }     // q and v: skip the k slice
      if (gemm_tc_supported(g)) a = g;
    }
    if ((e = linear(c, "lora_down_bwd", a))) return e;
  }
  // G_A = dh^T u (every qkv target in one pass over u) and G_B = (alpha/r) dy^T h of each target, per
  // group (Eq. 4-7): one batch, i.e. one pair of launches where the tensor-core path applies
  { LoraGradJob jobs[4];
    int nj = 0;
    LoraGradJob& ja = jobs[nj++];
    ja.Z = u; ja.ldz = d; ja.zcol0 = 0; ja.C = d; ja.Wt = c->g_dhcat; ja.ldwt = ext; ja.wcol0 = 0; ja.r = c->r; ja.rp = c->rp;
    ja.nt = c->nq; ja.scale = 1.0f; ja.out = gbase; ja.out_group_stride = gstride; ja.out_target_stride = (int64_t)2 * c->r * d;
    ja.out_sj = d; ja.out_sc = 1;
    for (int t = 0; t < c->nq; ++t) {
      LoraGradJob& jb = jobs[nj++];
      jb.Z = c->g_dqkv; jb.ldz = 3 * d; jb.zcol0 = c->slice_idx[t] * d; jb.C = d; jb.Wt = hcat; jb.ldwt = ext; jb.wcol0 = t * c->rp;
      jb.r = c->r; jb.rp = c->rp; jb.nt = 1; jb.scale = c->scale; jb.out = gbase + (size_t)t * 2 * c->r * d + (size_t)c->r * d;
      jb.out_group_stride = gstride; jb.out_target_stride = 0; jb.out_sj = 1; jb.out_sc = c->r;
    }
    Scope s(c, "lora_grad", 2);
    if ((e = lora_grad_batch(c->dt, jobs, nj, M, rpg, c->grad_scratch, c->grad_scratch_floats, c->st, c->status, c->tc))) return e; }
  if (dx) {
    GemmArgs a = base_args(c, c->g_dqkv, 3 * d, f.qkvwT, 3 * d, c->g_du, d, M, d, 3 * d);
    a.rows_per_group = rpg;
    a.Xe = c->g_dhcat; a.ldxe = ext; a.We = grp(k.AcatT, (size_t)d * ext); a.ldwe = ext; a.Ke = c->ke; a.we_grouped = grouped;
    if ((e = linear(c, "lora_linear_bwd", a))) return e;
    if ((e = norm_backward(c, M, c->g_du, at(b.x_in, d), f.ln1g, atf(b.mean1), atf(b.rstd1), c->g_dxmid, dx))) return e;
  }
  return cudaSuccess;
}

cudaError_t run_optimizer(splitlora_ctx* c, bool client) {
  OptArgs o;
  o.optimizer = c->cfg.optimizer; o.lr = client ? c->cfg.lr_client : c->cfg.lr_server;
  o.beta1 = c->cfg.beta1; o.beta2 = c->cfg.beta2; o.eps = c->cfg.adam_eps; o.wd = c->cfg.weight_decay;
  int64_t step = client ? ++c->client_steps : ++c->server_steps;
  o.bc1 = (float)(1.0 - std::pow((double)c->cfg.beta1, (double)step));
  o.bc2 = (float)(1.0 - std::pow((double)c->cfg.beta2, (double)step));
  Scope s(c, "optimizer", 1);
  if (client) return optimizer_step(c->cp, c->cg, c->cm, c->cv, (int64_t)c->K * c->Pc, o, c->st);
  return optimizer_step(c->sp, c->sg, c->sm, c->sv, c->Ps, o, c->st);
}

int check_ready(splitlora_ctx* c) {
  if (!c) return SPLITLORA_ERR_ARG;
  if (!c->ws) return fail(c, SPLITLORA_ERR_WORKSPACE, "no workspace bound");
  if (!all_frozen_bound(c)) return fail(c, SPLITLORA_ERR_STATE, "not every frozen tensor is bound");
  return SPLITLORA_OK;
}

float* adapter_ptr(splitlora_ctx* c, float* client_base, float* server_base, int side, int client, int layer,
                   uint32_t target, int* rc) {
  *rc = SPLITLORA_OK;
  int t = -1;
  for (int i = 0; i < c->n_targets; ++i) if (c->target_bit[i] == target) t = i;
  if (t < 0) { *rc = fail(c, SPLITLORA_ERR_ARG, "target is not an adapted slice"); return nullptr; }
  if (side == SPLITLORA_SIDE_CLIENT) {
    if (client < 0 || client >= c->K || layer < 0 || layer >= cut_of(c, client)) { *rc = fail(c, SPLITLORA_ERR_ARG, "client/layer out of range"); return nullptr; }
    return client_base + (size_t)client * c->Pc + (size_t)layer * c->per_layer + (size_t)t * 2 * c->r * c->d;
  }
  if (side == SPLITLORA_SIDE_SERVER) {
    if (layer < c->cmin || layer >= c->L) { *rc = fail(c, SPLITLORA_ERR_ARG, "layer out of range"); return nullptr; }
    return server_base + (size_t)(layer - c->cmin) * c->per_layer + (size_t)t * 2 * c->r * c->d;
  }
  *rc = fail(c, SPLITLORA_ERR_ARG, "bad side");
  return nullptr;
}

}  // namespace

// =============================================================================================
// C ABI
// =============================================================================================
extern "C" {

int splitlora_create(const splitlora_config* cfg, void* cuda_stream, splitlora_ctx** out) {
  if (!out) return SPLITLORA_ERR_ARG;
  *out = nullptr;
  std::string why;
  int rc = validate(cfg, &why);
  if (rc) return rc;
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return SPLITLORA_ERR_CUDA;
  if (prop.major != 10) return SPLITLORA_ERR_ARCH;
  if (gemm_tc_init() != 0) return SPLITLORA_ERR_CUDA;
  splitlora_ctx* c = new splitlora_ctx();
  c->cfg = *cfg;
  c->st = (cudaStream_t)cuda_stream;
  derive(c);
  *out = c;
  return SPLITLORA_OK;
}

int splitlora_destroy(splitlora_ctx* c) {
  if (!c) return SPLITLORA_ERR_ARG;
  for (auto& r : c->prof_recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  for (auto& e : c->event_pool) cudaEventDestroy(e);
  delete c;
  return SPLITLORA_OK;
}

int splitlora_workspace_bytes(const splitlora_config* cfg, size_t* bytes) {
  if (!bytes) return SPLITLORA_ERR_ARG;
  std::string why;
  int rc = validate(cfg, &why);
  if (rc) return rc;
  splitlora_ctx tmp;
  tmp.cfg = *cfg;
  derive(&tmp);
  *bytes = plan(&tmp, nullptr);
  return SPLITLORA_OK;
}

int splitlora_bind_workspace(splitlora_ctx* c, void* dev, size_t bytes) {
  if (!c || !dev) return SPLITLORA_ERR_ARG;
  if (reinterpret_cast<uintptr_t>(dev) & 255u) return fail(c, SPLITLORA_ERR_ALIGN, "workspace must be 256-byte aligned");
  size_t need = plan(c, nullptr);
  if (bytes < need) return fail(c, SPLITLORA_ERR_WORKSPACE, "workspace too small");
  plan(c, (char*)dev);
  c->ws = (char*)dev; c->ws_bytes = bytes;
  c->n_bound = 0;
  // zero: status, adapters, gradients, moments, and the padded compute copies
  CK(c, cudaMemsetAsync(c->status, 0, 256 * 3, c->st));
  for (float* p : {c->cp, c->cg, c->cm, c->cv}) CK(c, cudaMemsetAsync(p, 0, (size_t)c->K * c->Pc * 4, c->st));
  for (float* p : {c->sp, c->sg, c->sm, c->sv}) CK(c, cudaMemsetAsync(p, 0, (size_t)c->Ps * 4, c->st));
  for (int l = 0; l < c->L; ++l) {
    const size_t es = c->es, d = c->d, ext = c->ext;
    for (int side = 0; side < 2; ++side) {
      if (side == 0 ? l >= c->cut : l < c->cmin) continue;
      const size_t G = side == 0 ? c->K : 1;
      const LayerBuf::Copies& k = side == 0 ? c->lb[l].cl : c->lb[l].sv;
      CK(c, cudaMemsetAsync(k.Acat, 0, G * ext * d * es, c->st));
      CK(c, cudaMemsetAsync(k.AcatT, 0, G * ext * d * es, c->st));
      CK(c, cudaMemsetAsync(k.Bext, 0, G * 3 * d * ext * es, c->st));
      CK(c, cudaMemsetAsync(k.BextT, 0, G * 3 * d * ext * es, c->st));
      if (c->has_o)
        for (void* p : {k.AcatO, k.AcatOT, k.BextO, k.BextOT})
          CK(c, cudaMemsetAsync(p, 0, G * (size_t)c->ext_o * d * es, c->st));
    }
  }
  if (c->llama) {  // (cos, sin) of t * theta^(-2j/dh), evaluated in double
    const int half = c->d / c->cfg.n_head / 2, T = c->cfg.seq;
    c->rope_host.resize((size_t)T * half * 2);
    for (int t = 0; t < T; ++t)
      for (int j = 0; j < half; ++j) {
        const double ang = (double)t * std::pow((double)c->cfg.rope_theta, -2.0 * j / (2.0 * half));
        c->rope_host[((size_t)t * half + j) * 2] = (float)std::cos(ang);
        c->rope_host[((size_t)t * half + j) * 2 + 1] = (float)std::sin(ang);
      }
    CK(c, cudaMemcpyAsync(c->rope_table, c->rope_host.data(), c->rope_host.size() * 4, cudaMemcpyHostToDevice, c->st));
  }
  CK(c, cudaMemsetAsync(c->wteT, 0, (size_t)c->d * c->Vpad * c->es, c->st));
  c->client_copies_dirty = c->server_copies_dirty = true;
  c->have_client_fwd = false;
  c->round_index = c->server_steps = c->client_steps = 0;
  c->client_cut.clear();
  return SPLITLORA_OK;
}

int splitlora_bind_frozen(splitlora_ctx* c, const char* name, const void* dev, size_t bytes) {
  if (!c || !name || !dev) return SPLITLORA_ERR_ARG;
  if (!c->ws) return fail(c, SPLITLORA_ERR_WORKSPACE, "bind the workspace first");
  if (!aligned16(dev)) return fail(c, SPLITLORA_ERR_ALIGN, std::string(name) + " is not 16-byte aligned");
  const size_t es = c->es, d = c->d, F = c->F;
  auto expect = [&](size_t elems) { return bytes == elems * es; };
  auto bad_size = [&]() { return fail(c, SPLITLORA_ERR_ARG, std::string("wrong byte size for ") + name); };
  auto set = [&](const void** slot) { if (!*slot) c->n_bound++; *slot = dev; };
  std::string n(name);
  if (n == "wte" || (c->llama && n == "head.w")) {
    if (!expect((size_t)c->V * d)) return bad_size();
    if (n == "wte") set(&c->wte);
    if (n == "head.w" || !c->llama) {      // the head: tied to wte unless the architecture has its own
      if (c->llama) set(&c->headw); else c->headw = dev;
      Scope s(c, "transpose", 1);
      CK(c, transpose(c->dt, dev, c->V, c->d, c->wteT, c->Vpad, c->st));
    }
    return SPLITLORA_OK;
  }
  if (n == "lnf.g") { if (!expect(d)) return bad_size(); set(&c->lnfg); return SPLITLORA_OK; }
  if (!c->llama) {
    if (n == "wpe") { if (!expect((size_t)c->cfg.max_seq * d)) return bad_size(); set(&c->wpe); return SPLITLORA_OK; }
    if (n == "lnf.b") { if (!expect(d)) return bad_size(); set(&c->lnfb); return SPLITLORA_OK; }
  }
  int l = -1; char rest[64];
  if (sscanf(name, "h.%d.%63s", &l, rest) != 2 || l < 0 || l >= c->L) return fail(c, SPLITLORA_ERR_ARG, std::string("unknown tensor ") + name);
  FrozenLayer& f = c->fl[l];
  std::string r(rest);
  struct Ent { const char* nm; const void** slot; size_t elems; void* tr; int rows, cols; bool gpt, llama; };
  Ent ents[] = {
      {"ln1.g", &f.ln1g, d, nullptr, 0, 0, true, true}, {"ln1.b", &f.ln1b, d, nullptr, 0, 0, true, false},
      {"attn.qkv.w", &f.qkvw, 3 * d * d, f.qkvwT, 3 * c->d, c->d, true, true},
      {"attn.qkv.b", &f.qkvb, 3 * d, nullptr, 0, 0, true, false},
      {"attn.proj.w", &f.projw, d * d, f.projwT, c->d, c->d, true, true},
      {"attn.proj.b", &f.projb, d, nullptr, 0, 0, true, false},
      {"ln2.g", &f.ln2g, d, nullptr, 0, 0, true, true}, {"ln2.b", &f.ln2b, d, nullptr, 0, 0, true, false},
      {"mlp.fc1.w", &f.fc1w, F * d, f.fc1wT, c->F, c->d, true, false}, {"mlp.fc1.b", &f.fc1b, F, nullptr, 0, 0, true, false},
      {"mlp.fc2.w", &f.fc2w, d * F, f.fc2wT, c->d, c->F, true, false}, {"mlp.fc2.b", &f.fc2b, d, nullptr, 0, 0, true, false},
      {"mlp.gate_up.w", &f.fc1w, 2 * F * d, f.fc1wT, 2 * c->F, c->d, false, true},
      {"mlp.down.w", &f.fc2w, d * F, f.fc2wT, c->d, c->F, false, true}};
  for (auto& e : ents) {
    if (r == e.nm && (c->llama ? e.llama : e.gpt)) {
      if (!expect(e.elems)) return bad_size();
      set(e.slot);
      if (e.tr) {
        Scope s(c, "transpose", 1);
        CK(c, transpose(c->dt, dev, e.rows, e.cols, e.tr, e.rows, c->st));
      }
      return SPLITLORA_OK;
    }
  }
  return fail(c, SPLITLORA_ERR_ARG, std::string("unknown tensor ") + name);
}

int splitlora_set_adapter(splitlora_ctx* c, int side, int client, int layer, uint32_t target, const float* A,
                          const float* B) {
  if (!c) return SPLITLORA_ERR_ARG;
  if (!c->ws) return fail(c, SPLITLORA_ERR_WORKSPACE, "no workspace bound");
  int rc;
  float* p = adapter_ptr(c, c->cp, c->sp, side, client, layer, target, &rc);
  if (!p) return rc;
  const size_t n = (size_t)c->r * c->d * 4;
  if (A) CK(c, cudaMemcpyAsync(p, A, n, cudaMemcpyDeviceToDevice, c->st));
  if (B) CK(c, cudaMemcpyAsync(p + (size_t)c->r * c->d, B, n, cudaMemcpyDeviceToDevice, c->st));
  (side == SPLITLORA_SIDE_CLIENT ? c->client_copies_dirty : c->server_copies_dirty) = true;
  return SPLITLORA_OK;
}

static int get_pair(splitlora_ctx* c, float* cb, float* sb, int side, int client, int layer, uint32_t target,
                    float* A, float* B) {
  if (!c) return SPLITLORA_ERR_ARG;
  if (!c->ws) return fail(c, SPLITLORA_ERR_WORKSPACE, "no workspace bound");
  int rc;
  float* p = adapter_ptr(c, cb, sb, side, client, layer, target, &rc);
  if (!p) return rc;
  const size_t n = (size_t)c->r * c->d * 4;
  if (A) CK(c, cudaMemcpyAsync(A, p, n, cudaMemcpyDeviceToDevice, c->st));
  if (B) CK(c, cudaMemcpyAsync(B, p + (size_t)c->r * c->d, n, cudaMemcpyDeviceToDevice, c->st));
  return SPLITLORA_OK;
}

int splitlora_get_adapter(splitlora_ctx* c, int side, int client, int layer, uint32_t target, float* A, float* B) {
  return get_pair(c, c ? c->cp : nullptr, c ? c->sp : nullptr, side, client, layer, target, A, B);
}
int splitlora_get_adapter_grad(splitlora_ctx* c, int side, int client, int layer, uint32_t target, float* dA, float* dB) {
  return get_pair(c, c ? c->cg : nullptr, c ? c->sg : nullptr, side, client, layer, target, dA, dB);
}
int splitlora_get_opt_state(splitlora_ctx* c, int side, int client, int layer, uint32_t target, float* mA, float* vA,
                            float* mB, float* vB) {
  int rc = get_pair(c, c ? c->cm : nullptr, c ? c->sm : nullptr, side, client, layer, target, mA, mB);
  if (rc) return rc;
  return get_pair(c, c->cv, c->sv, side, client, layer, target, vA, vB);
}
int splitlora_set_opt_state(splitlora_ctx* c, int side, int client, int layer, uint32_t target, const float* mA,
                            const float* vA, const float* mB, const float* vB) {
  if (!c) return SPLITLORA_ERR_ARG;
  if (!c->ws) return fail(c, SPLITLORA_ERR_WORKSPACE, "no workspace bound");
  int rc;
  float* pm = adapter_ptr(c, c->cm, c->sm, side, client, layer, target, &rc);
  if (!pm) return rc;
  float* pv = adapter_ptr(c, c->cv, c->sv, side, client, layer, target, &rc);
  const size_t n = (size_t)c->r * c->d * 4, o = (size_t)c->r * c->d;
  if (mA) CK(c, cudaMemcpyAsync(pm, mA, n, cudaMemcpyDeviceToDevice, c->st));
  if (mB) CK(c, cudaMemcpyAsync(pm + o, mB, n, cudaMemcpyDeviceToDevice, c->st));
  if (vA) CK(c, cudaMemcpyAsync(pv, vA, n, cudaMemcpyDeviceToDevice, c->st));
  if (vB) CK(c, cudaMemcpyAsync(pv + o, vB, n, cudaMemcpyDeviceToDevice, c->st));
  return SPLITLORA_OK;
}
int splitlora_get_counters(splitlora_ctx* c, int64_t* round_index, int64_t* server_steps, int64_t* client_steps) {
  if (!c) return SPLITLORA_ERR_ARG;
  if (round_index) *round_index = c->round_index;
  if (server_steps) *server_steps = c->server_steps;
  if (client_steps) *client_steps = c->client_steps;
  return SPLITLORA_OK;
}
int splitlora_set_counters(splitlora_ctx* c, int64_t round_index, int64_t server_steps, int64_t client_steps) {
  if (!c || round_index < 0 || server_steps < 0 || client_steps < 0) return SPLITLORA_ERR_ARG;
  c->round_index = round_index; c->server_steps = server_steps; c->client_steps = client_steps;
  return SPLITLORA_OK;
}

// ---- Algorithm 1 ---------------------------------------------------------------------------

int splitlora_client_fwd(splitlora_ctx* c, const int32_t* tokens, void* act_out) {
  int rc = check_ready(c);
  if (rc) return rc;
  if (!tokens || !act_out) return fail(c, SPLITLORA_ERR_ARG, "null pointer");
  if (!aligned16(tokens) || !aligned16(act_out)) return fail(c, SPLITLORA_ERR_ALIGN, "tokens / act_out not 16-byte aligned");
  if (c->client_copies_dirty) { CK(c, refresh_side(c, true)); c->client_copies_dirty = false; }
  { Scope s(c, "embed", 1);
    CK(c, embed(c->dt, tokens, c->wte, c->wpe, c->emb, c->M, c->cfg.seq, c->d, c->V, c->st)); }
  const void* x = c->emb;
  for (int l = 0; l < c->cut; ++l) {
    // clients whose last block this is hand their output off: written in place when that is everybody,
    // else copied out of the block's output buffer (the others go on from there)
    const Span sp = client_span(c, l);
    const bool all_finish = first_client_above(c, l + 1) == c->K && sp.client0 == 0;
    void* out = all_finish ? act_out : c->lb[l].x_out;
    CK(c, block_forward(c, l, sp, x, out));
    if (!all_finish) CK(c, copy_client_rows(c, out, act_out, sp.client0, first_client_above(c, l + 1)));
    x = out;
  }
  c->have_client_fwd = true;
  return SPLITLORA_OK;
}

int splitlora_server_step(splitlora_ctx* c, const void* act_in, const int32_t* labels, void* act_grad_out,
                          float* loss_out) {
  int rc = check_ready(c);
  if (rc) return rc;
  if (!act_in || !labels || !act_grad_out) return fail(c, SPLITLORA_ERR_ARG, "null pointer");
  if (!aligned16(act_in) || !aligned16(labels) || !aligned16(act_grad_out)) return fail(c, SPLITLORA_ERR_ALIGN, "buffer not 16-byte aligned");
  if (c->server_copies_dirty) { CK(c, refresh_side(c, false)); c->server_copies_dirty = false; }
  const int M = c->M, d = c->d;
  // forward over the concatenated batch S^t (Eq. 3).  With clients cut at different depths the batch of
  // block l is the prefix of clients that have handed off by then; a client's rows join the stream of the
  // block below its entry point (a copy of its hand-off), so every block reads one contiguous buffer.
  const bool uni = uniform_cut(c);
  const int first = uni ? c->cut : c->cmin;        // first block the server runs
  const void* x = act_in;
  for (int l = first; l < c->L; ++l) {
    if (!uni) {
      CK(c, copy_client_rows(c, act_in, c->lb[l - 1].x_out, first_client_above(c, l - 1), first_client_above(c, l)));
      x = c->lb[l - 1].x_out;
    }
    CK(c, block_forward(c, l, server_span(c, l), x, c->lb[l].x_out));
    x = c->lb[l].x_out;
  }
  if (!uni) {   // clients that hand off above the last block enter at the final norm
    CK(c, copy_client_rows(c, act_in, c->lb[c->L - 1].x_out, first_client_above(c, c->L - 1), c->K));
    x = c->lb[c->L - 1].x_out;
  }
  CK(c, norm_forward(c, M, x, c->lnfg, c->lnfb, c->xf, c->meanf, c->rstdf));
  { GemmArgs a = base_args(c, c->xf, d, c->headw, d, c->logits, c->Vpad, M, c->Vpad, d);
    a.w_rows = c->V;
    CK(c, linear(c, "head_fwd", a)); }
  { Scope s(c, "cross_entropy", 3);
    CK(c, cross_entropy(c->dt, c->logits, c->Vpad, labels, M, c->V, c->row_loss, c->n_valid, c->loss_dev,
                        (int)c->loss_normalizer, c->st)); }
  // backward: head, final norm, blocks L-1 .. first
  { GemmArgs a = base_args(c, c->logits, c->Vpad, c->wteT, c->Vpad, c->g_a, d, M, d, c->Vpad);
    CK(c, linear(c, "head_bwd", a)); }
  void* cur = (uni && c->cut == c->L) ? act_grad_out : c->g_b;     // no server block: this is dL/dS already
  CK(c, norm_backward(c, M, c->g_a, x, c->lnfg, c->meanf, c->rstdf, nullptr, cur));
  void* other = c->g_a;
  for (int l = c->L - 1; l >= first; --l) {
    // rows of the clients that entered above block l hold their dL/ds_i now: hand them back
    if (!uni) CK(c, copy_client_rows(c, cur, act_grad_out, first_client_above(c, l), first_client_above(c, l + 1)));
    void* dst = (uni && l == first) ? act_grad_out : other;
    CK(c, block_backward(c, l, server_span(c, l), cur, dst));
    other = cur; cur = dst;
  }
  if (!uni) CK(c, copy_client_rows(c, cur, act_grad_out, 0, first_client_above(c, c->cmin)));
  // Eq. 4-5: server update
  if (!c->defer_server_update) {
    CK(c, run_optimizer(c, false));
    c->server_copies_dirty = true;
  }
  if (loss_out) {
    CK(c, cudaMemcpyAsync(loss_out, c->loss_dev, 4, cudaMemcpyDeviceToHost, c->st));
    CK(c, cudaStreamSynchronize(c->st));
    int code = 0;
    CK(c, cudaMemcpy(&code, c->status, 4, cudaMemcpyDeviceToHost));
    if (code) return fail(c, SPLITLORA_ERR_TIMEOUT, "a bounded device wait expired (code " + std::to_string(code) + ")");
  }
  return SPLITLORA_OK;
}

int splitlora_client_bwd(splitlora_ctx* c, const void* act_grad_in) {
  int rc = check_ready(c);
  if (rc) return rc;
  if (!act_grad_in) return fail(c, SPLITLORA_ERR_ARG, "null pointer");
  if (!aligned16(act_grad_in)) return fail(c, SPLITLORA_ERR_ALIGN, "act_grad_in not 16-byte aligned");
  if (!c->have_client_fwd) return fail(c, SPLITLORA_ERR_STATE, "client_bwd needs a preceding client_fwd");
  // With one cut for all, the hand-off gradient is read in place.  Otherwise each client's rows are copied
  // into the stream of gradients where its deepest block begins.
  const bool uni = uniform_cut(c);
  void* bufs[2] = {c->g_a, c->g_b};
  const void* cur = uni ? act_grad_in : bufs[1];
  int which = 0;
  for (int l = c->cut - 1; l >= 0; --l) {
    const Span sp = client_span(c, l);
    if (!uni) CK(c, copy_client_rows(c, act_grad_in, (void*)cur, sp.client0, first_client_above(c, l + 1)));
    void* dst = (l == 0) ? nullptr : bufs[which];
    CK(c, block_backward(c, l, sp, cur, dst));
    cur = dst; which ^= 1;
  }
  CK(c, run_optimizer(c, true));   // Eq. 6-7, all K clients in one launch
  c->client_copies_dirty = true;
  c->have_client_fwd = false;
  return SPLITLORA_OK;
}

// w_i = |D_i| / total, total = the local sum or, when the clients are spread over devices, |D| of all of them
static int aggregation_weights(splitlora_ctx* c, const int64_t* counts, double total_override, float* w) {
  if (!c) return SPLITLORA_ERR_ARG;
  if (!c->ws) return fail(c, SPLITLORA_ERR_WORKSPACE, "no workspace bound");
  if (!counts) return fail(c, SPLITLORA_ERR_ARG, "null counts");
  double total = 0.0;
  for (int i = 0; i < c->K; ++i) {
    if (counts[i] < 0) return fail(c, SPLITLORA_ERR_COUNTS, "negative sample count");
    total += (double)counts[i];
  }
  if (total_override > 0.0) {
    if (total > total_override) return fail(c, SPLITLORA_ERR_COUNTS, "local counts exceed the global total");
    total = total_override;
  }
  if (!(total > 0.0)) return fail(c, SPLITLORA_ERR_COUNTS, "all sample counts are zero");
  for (int i = 0; i < c->K; ++i) w[i] = (float)((double)counts[i] / total);
  return SPLITLORA_OK;
}

int splitlora_set_client_ranks(splitlora_ctx* c, const int32_t* ranks) {
  if (!c) return SPLITLORA_ERR_ARG;
  if (!c->ws) return fail(c, SPLITLORA_ERR_WORKSPACE, "no workspace bound");
  if (!ranks) { c->client_rank.clear(); return SPLITLORA_OK; }
  for (int i = 0; i < c->K; ++i)
    if (ranks[i] < 1 || ranks[i] > c->r) return fail(c, SPLITLORA_ERR_ARG, "client rank outside [1, lora_r]");
  c->client_rank.assign(ranks, ranks + c->K);
  // parameters and both moments: what a client does not have is zero from here on (its gradient is
  // exactly zero, so the updates keep it there)
  float* arenas[3] = {c->cp, c->cm, c->cv};
  for (float* a : arenas) CK(c, rank_mask(a, c->K, c->Pc, c->r, c->d, c->client_rank.data(), c->st));
  c->launches += 3;
  c->client_copies_dirty = true;
  return SPLITLORA_OK;
}

int splitlora_aggregate(splitlora_ctx* c, const int64_t* counts) {
  float w[AGG_MAX_CLIENTS];
  int rc = aggregation_weights(c, counts, 0.0, w);
  if (rc) return rc;
  if (uniform_cut(c)) {
    Scope s(c, "aggregate", 1);
    CK(c, aggregate(c->cp, c->K, c->Pc, w, c->st));
  } else {
    // Eq. 8-9 per block over the clients that hold it (a suffix of the clients), weights renormalised
    // over those holders; a block with a single holder stays as it is
    for (int l = 0; l < c->cut; ++l) {
      const int h0 = first_client_above(c, l), nh = c->K - h0;
      if (nh < 2) continue;
      double tot = 0.0;
      for (int i = h0; i < c->K; ++i) tot += (double)counts[i];
      if (!(tot > 0.0)) return fail(c, SPLITLORA_ERR_COUNTS, "all sample counts of a block's holders are zero");
      float wl[AGG_MAX_CLIENTS];
      for (int i = 0; i < nh; ++i) wl[i] = (float)((double)counts[h0 + i] / tot);
      Scope s(c, "aggregate", 1);
      CK(c, aggregate(c->cp + (size_t)h0 * c->Pc + (size_t)l * c->per_layer, nh, c->per_layer, wl, c->st, c->Pc));
    }
  }
  // clients of lower rank keep only their own components of the (zero-padded) average
  if (!c->client_rank.empty()) {
    Scope s(c, "aggregate", 1);
    CK(c, rank_mask(c->cp, c->K, c->Pc, c->r, c->d, c->client_rank.data(), c->st));
  }
  c->client_copies_dirty = true;
  return SPLITLORA_OK;
}

int splitlora_set_client_cuts(splitlora_ctx* c, const int32_t* cuts) {
  if (!c) return SPLITLORA_ERR_ARG;
  if (!c->ws) return fail(c, SPLITLORA_ERR_WORKSPACE, "no workspace bound");
  if (!cuts) { c->client_cut.clear(); return SPLITLORA_OK; }
  for (int i = 0; i < c->K; ++i) {
    if (cuts[i] < c->cmin || cuts[i] > c->cut) return fail(c, SPLITLORA_ERR_ARG, "client cut outside [cut_min, cut]");
    if (i > 0 && cuts[i] < cuts[i - 1]) return fail(c, SPLITLORA_ERR_ARG, "client cuts must be non-decreasing in the client index");
  }
  bool same = true;
  for (int i = 0; i < c->K; ++i) same = same && cuts[i] == c->cut;
  if (same) c->client_cut.clear(); else c->client_cut.assign(cuts, cuts + c->K);
  c->have_client_fwd = false;
  return SPLITLORA_OK;
}

// ---- hooks for sharding the clients over several devices --------------------------------------

int splitlora_aggregate_local_sum(splitlora_ctx* c, const int64_t* counts, int64_t total_count, float** sum_dev,
                                  int64_t* count) {
  if (!c || !sum_dev || !count) return SPLITLORA_ERR_ARG;
  if (total_count <= 0) return fail(c, SPLITLORA_ERR_COUNTS, "total_count must be positive");
  if (!uniform_cut(c)) return fail(c, SPLITLORA_ERR_UNSUPPORTED, "clients cut at different depths cannot be spread over devices");
  float w[AGG_MAX_CLIENTS];
  int rc = aggregation_weights(c, counts, (double)total_count, w);
  if (rc) return rc;
  { Scope s(c, "aggregate", 1);
    CK(c, aggregate_local_sum(c->cp, c->K, c->Pc, w, c->agg_sum, c->st)); }
  *sum_dev = c->agg_sum; *count = c->Pc;
  return SPLITLORA_OK;
}

int splitlora_aggregate_broadcast(splitlora_ctx* c) {
  if (!c) return SPLITLORA_ERR_ARG;
  if (!c->ws) return fail(c, SPLITLORA_ERR_WORKSPACE, "no workspace bound");
  { Scope s(c, "aggregate", c->client_rank.empty() ? 1 : 2);
    CK(c, aggregate_broadcast(c->agg_sum, c->K, c->Pc, c->cp, c->st));
    // the mask comes after the sum over devices: the sum holds every client's components
    if (!c->client_rank.empty()) CK(c, rank_mask(c->cp, c->K, c->Pc, c->r, c->d, c->client_rank.data(), c->st)); }
  c->client_copies_dirty = true;
  return SPLITLORA_OK;
}

int splitlora_set_loss_normalizer(splitlora_ctx* c, int64_t n_valid_global) {
  if (!c || n_valid_global < 0 || n_valid_global > 2147483647LL) return SPLITLORA_ERR_ARG;
  c->loss_normalizer = n_valid_global;
  return SPLITLORA_OK;
}

int splitlora_set_deferred_server_update(splitlora_ctx* c, int on) {
  if (!c) return SPLITLORA_ERR_ARG;
  c->defer_server_update = on != 0;
  return SPLITLORA_OK;
}

int splitlora_server_update(splitlora_ctx* c) {
  int rc = check_ready(c);
  if (rc) return rc;
  CK(c, run_optimizer(c, false));
  c->server_copies_dirty = true;
  return SPLITLORA_OK;
}

int splitlora_adapter_buffer(splitlora_ctx* c, int side, int kind, float** dev, int64_t* count) {
  if (!c || !dev || !count) return SPLITLORA_ERR_ARG;
  if (!c->ws) return fail(c, SPLITLORA_ERR_WORKSPACE, "no workspace bound");
  if (kind != 0 && kind != 1) return fail(c, SPLITLORA_ERR_ARG, "kind must be 0 (parameters) or 1 (gradients)");
  if (side == SPLITLORA_SIDE_CLIENT) { *dev = kind ? c->cg : c->cp; *count = (int64_t)c->K * c->Pc; }
  else if (side == SPLITLORA_SIDE_SERVER) { *dev = kind ? c->sg : c->sp; *count = c->Ps; }
  else return fail(c, SPLITLORA_ERR_ARG, "bad side");
  return SPLITLORA_OK;
}

int splitlora_adapters_changed(splitlora_ctx* c, int side) {
  if (!c) return SPLITLORA_ERR_ARG;
  if (side == SPLITLORA_SIDE_CLIENT) c->client_copies_dirty = true;
  else if (side == SPLITLORA_SIDE_SERVER) c->server_copies_dirty = true;
  else return fail(c, SPLITLORA_ERR_ARG, "bad side");
  return SPLITLORA_OK;
}

int splitlora_round(splitlora_ctx* c, const int32_t* tokens, const int32_t* labels, const int64_t* counts,
                    float* loss_out) {
  int rc = check_ready(c);
  if (rc) return rc;
  if (!counts) return fail(c, SPLITLORA_ERR_ARG, "null counts");
  if ((rc = splitlora_client_fwd(c, tokens, c->S))) return rc;
  if ((rc = splitlora_server_step(c, c->S, labels, c->dS, nullptr))) return rc;
  if ((rc = splitlora_client_bwd(c, c->dS))) return rc;
  c->round_index++;
  if (c->round_index % c->cfg.agg_interval == 0)
    if ((rc = splitlora_aggregate(c, counts))) return rc;
  if (loss_out) {
    CK(c, cudaMemcpyAsync(loss_out, c->loss_dev, 4, cudaMemcpyDeviceToHost, c->st));
    CK(c, cudaStreamSynchronize(c->st));
    int code = 0;
    CK(c, cudaMemcpy(&code, c->status, 4, cudaMemcpyDeviceToHost));
    if (code) return fail(c, SPLITLORA_ERR_TIMEOUT, "a bounded device wait expired (code " + std::to_string(code) + ")");
  }
  return SPLITLORA_OK;
}

int splitlora_round_compressed(splitlora_ctx* c, const int32_t* tokens, const int32_t* labels, const int64_t* counts,
                               uint8_t* codes, float* scales, float* loss_out) {
  int rc = check_ready(c);
  if (rc) return rc;
  if (!counts || !codes || !scales) return fail(c, SPLITLORA_ERR_ARG, "null pointer");
  const int n = c->dt == DT_BF16 ? 8 : 4;
  if (c->d % n != 0) return fail(c, SPLITLORA_ERR_ARG, "d_model is not a multiple of the codec's vector width");
  if (!aligned16(codes)) return fail(c, SPLITLORA_ERR_ALIGN, "codes not 16-byte aligned");
  const size_t Md = (size_t)c->M * (size_t)c->d;
  // what crosses the cut is codes + scales; the receiving side restores into the buffer it reads
  auto cross = [&](void* buf, uint8_t* q, float* sc) -> int {
    Scope s(c, "handoff_codec", 2);
    CK(c, handoff_quantize(c->dt, buf, c->M, c->d, q, sc, c->st));
    CK(c, handoff_dequantize(c->dt, q, sc, c->M, c->d, buf, c->st));
    return SPLITLORA_OK;
  };
  if ((rc = splitlora_client_fwd(c, tokens, c->S))) return rc;
  if ((rc = cross(c->S, codes, scales))) return rc;
  if ((rc = splitlora_server_step(c, c->S, labels, c->dS, nullptr))) return rc;
  if ((rc = cross(c->dS, codes + Md, scales + c->M))) return rc;
  if ((rc = splitlora_client_bwd(c, c->dS))) return rc;
  c->round_index++;
  if (c->round_index % c->cfg.agg_interval == 0)
    if ((rc = splitlora_aggregate(c, counts))) return rc;
  if (loss_out) {
    CK(c, cudaMemcpyAsync(loss_out, c->loss_dev, 4, cudaMemcpyDeviceToHost, c->st));
    CK(c, cudaStreamSynchronize(c->st));
    int code = 0;
    CK(c, cudaMemcpy(&code, c->status, 4, cudaMemcpyDeviceToHost));
    if (code) return fail(c, SPLITLORA_ERR_TIMEOUT, "a bounded device wait expired (code " + std::to_string(code) + ")");
  }
  return SPLITLORA_OK;
}

int splitlora_round_host(splitlora_ctx* c, const int32_t* tokens_host, const int32_t* labels_host,
                         const int64_t* counts, float* loss_out) {
  int rc = check_ready(c);
  if (rc) return rc;
  if (!tokens_host || !labels_host) return fail(c, SPLITLORA_ERR_ARG, "null pointer");
  CK(c, cudaMemcpyAsync(c->tok_dev, tokens_host, (size_t)c->M * 4, cudaMemcpyHostToDevice, c->st));
  CK(c, cudaMemcpyAsync(c->lab_dev, labels_host, (size_t)c->M * 4, cudaMemcpyHostToDevice, c->st));
  return splitlora_round(c, c->tok_dev, c->lab_dev, counts, loss_out);
}

int splitlora_loss_device(splitlora_ctx* c, const float** loss_dev) {
  if (!c || !loss_dev) return SPLITLORA_ERR_ARG;
  if (!c->ws) return fail(c, SPLITLORA_ERR_WORKSPACE, "no workspace bound");
  *loss_dev = c->loss_dev;
  return SPLITLORA_OK;
}

const char* splitlora_last_error(const splitlora_ctx* c) { return c ? c->err.c_str() : "null context"; }

int splitlora_device_status(splitlora_ctx* c, int32_t* code) {
  if (!c || !code) return SPLITLORA_ERR_ARG;
  if (!c->ws) return fail(c, SPLITLORA_ERR_WORKSPACE, "no workspace bound");
  CK(c, cudaStreamSynchronize(c->st));
  CK(c, cudaMemcpy(code, c->status, 4, cudaMemcpyDeviceToHost));
  return SPLITLORA_OK;
}

int splitlora_launch_count(const splitlora_ctx* c, int64_t* launches) {
  if (!c || !launches) return SPLITLORA_ERR_ARG;
  *launches = c->launches;
  return SPLITLORA_OK;
}

int splitlora_profile_enable(splitlora_ctx* c, int on) {
  if (!c) return SPLITLORA_ERR_ARG;
  c->prof_on = on < 0 || on > 2 ? 1 : on;
  return SPLITLORA_OK;
}

int splitlora_profile_report(splitlora_ctx* c, char (*names)[48], int64_t* launches, double* ms, int cap, int* n) {
  if (!c || !n) return SPLITLORA_ERR_ARG;
  CK(c, cudaStreamSynchronize(c->st));
  std::vector<double> tot(c->prof_names.size(), 0.0);
  std::vector<int64_t> cnt(c->prof_names.size(), 0);
  for (auto& r : c->prof_recs) {
    float t = 0.f;
    CK(c, cudaEventElapsedTime(&t, r.a, r.b));
    tot[r.cls] += t; cnt[r.cls] += 1;
    c->event_pool.push_back(r.a); c->event_pool.push_back(r.b);
  }
  c->prof_recs.clear();
  *n = (int)c->prof_names.size();
  for (int i = 0; i < *n && i < cap; ++i) {
    if (names) { std::strncpy(names[i], c->prof_names[i].c_str(), 47); names[i][47] = 0; }
    if (launches) launches[i] = cnt[i];
    if (ms) ms[i] = tot[i];
  }
  return SPLITLORA_OK;
}

}  // extern "C"
