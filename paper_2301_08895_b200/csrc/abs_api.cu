// C ABI of the ABS round loop: argument checks, workspace carving, per-round kernel sequence.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"
#include "ctl.cuh"
#include "simt.cuh"

using namespace absb;

namespace {

thread_local std::string g_err;

int fail(int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  g_err = buf;
  return code;
}

struct Carver {
  size_t off = 0;
  size_t take(size_t bytes) {
    const size_t o = off;
    off = round_up_sz(off + bytes, 256);
    return o;
  }
};

// Byte offsets of everything inside the workspace.
struct Layout {
  int n_layers = 0, RB = 0, rows_cap = 0, P = 0, n_tiles_cap = 0;
  size_t esz = 4;                       // bytes per stored element (4 or 2)
  size_t d = 0, d_pad = 0;
  size_t w_off[ABS_MAX_LAYERS] = {};    // element offset of W_l inside the padded vector
  size_t w_src[ABS_MAX_LAYERS] = {};    // element offset of W_l inside the caller's vector
  size_t st, c, version, job, sel, sel_tau, sel_row0, loss, row_loss, row_idx, tile_slot;
  size_t master, ring, G, logits;
  size_t act[ABS_MAX_LAYERS + 1], delta[ABS_MAX_LAYERS + 1];
  size_t tr_K, tr_R, tr_theta, tr_T, tr_loss, tr_comm, tr_sel_off, tr_rst_off;
  size_t tr_sel_id, tr_sel_tau, tr_sel_loss, tr_rst_id;
  size_t data_X, data_y;
  size_t total = 0;
};

int check_model(const abs_model_desc* m, int W, int S) {
  if (!m) return fail(ABS_EINVAL, "model is null");
  if (m->kind != ABS_LSQ && m->kind != ABS_SOFTMAX && m->kind != ABS_MLP)
    return fail(ABS_EUNSUPPORTED, "unknown model kind %d", m->kind);
  if (m->dtype != ABS_FP32 && m->dtype != ABS_BF16_FP32MASTER)
    return fail(ABS_EUNSUPPORTED, "unknown dtype %d", m->dtype);
  if (m->n_layers < 1 || m->n_layers > ABS_MAX_LAYERS)
    return fail(ABS_EINVAL, "n_layers %d outside [1, %d]", m->n_layers, ABS_MAX_LAYERS);
  if ((m->kind == ABS_LSQ || m->kind == ABS_SOFTMAX) && m->n_layers != 1)
    return fail(ABS_EINVAL, "this model kind has exactly one layer");
  for (int l = 0; l <= m->n_layers; ++l)
    if (m->dims[l] < 1 || m->dims[l] > (1 << 20)) return fail(ABS_EINVAL, "dims[%d] = %d", l, m->dims[l]);
  if (m->kind == ABS_LSQ && m->dims[1] != 1) return fail(ABS_EINVAL, "least squares needs dims = {d, 1}");
  if (m->kind != ABS_LSQ && (m->dims[m->n_layers] < 2 || m->dims[m->n_layers] > 64))
    return fail(ABS_EINVAL, "class count %d outside [2, 64]", m->dims[m->n_layers]);
  if (m->batch < 1 || m->batch > 1024) return fail(ABS_EINVAL, "batch %d outside [1, 1024]", m->batch);
  if (m->max_rounds < 1) return fail(ABS_EINVAL, "max_rounds %d < 1", m->max_rounds);
  if (m->n_samples < 1 || m->n_samples > 0x7fffffffLL) return fail(ABS_EINVAL, "n_samples out of range");
  if (W < 1 || W > ABS_MAX_WORKERS) return fail(ABS_EINVAL, "W %d outside [1, %d]", W, ABS_MAX_WORKERS);
  if (m->n_samples < W) return fail(ABS_EINVAL, "fewer samples than workers");
  if (S < 0 || S > ABS_MAX_BOUND) return fail(ABS_EINVAL, "staleness_bound %d outside [0, %d]", S, ABS_MAX_BOUND);
  return ABS_OK;
}

void make_layout(const abs_model_desc* m, int W, int S, Layout* L) {
  L->n_layers = m->n_layers;
  L->esz = m->dtype == ABS_FP32 ? 4 : 2;
  const bool lsq = m->kind == ABS_LSQ;
  // padded parameter vector: each layer's [W | b] block starts on a 64-element boundary
  size_t off = 0, src = 0;
  for (int l = 0; l < m->n_layers; ++l) {
    L->w_off[l] = off;
    L->w_src[l] = src;
    const size_t n = lsq ? (size_t)m->dims[0] : (size_t)m->dims[l] * m->dims[l + 1] + m->dims[l + 1];
    off = round_up_sz(off + n, 64);
    src += n;
  }
  L->d = src;
  L->d_pad = round_up_sz(off, 256);
  L->RB = lsq ? m->batch : 64;
  const int groups = (W < S + 1) ? W : S + 1;
  L->rows_cap = round_up(W * m->batch, L->RB) + groups * L->RB;
  L->n_tiles_cap = L->rows_cap / L->RB;
  if (lsq) {
    L->P = 0;
  } else {
    // split count of the row reduction in the weight-gradient kernels
    size_t tiles = 0;
    for (int l = 0; l < m->n_layers; ++l)
      tiles = std::max(tiles, (size_t)((m->dims[l] + 1 + TM - 1) / TM) * ((m->dims[l + 1] + TN - 1) / TN));
    int P = (int)((296 + tiles - 1) / tiles);
    P = std::min(P, std::max(1, W * m->batch / 128));
    L->P = std::max(1, std::min(P, 16));
  }
  Carver cv;
  L->st = cv.take(sizeof(DevState));
  L->c = cv.take(sizeof(u64) * W);
  L->version = cv.take(4 * W);
  L->job = cv.take(4 * W);
  L->sel = cv.take(4 * W);
  L->sel_tau = cv.take(4 * W);
  L->sel_row0 = cv.take(4 * W);
  L->loss = cv.take(4 * W);
  L->row_loss = cv.take(4 * (size_t)L->rows_cap);
  L->row_idx = cv.take(4 * (size_t)L->rows_cap);
  L->tile_slot = cv.take(4 * (size_t)L->n_tiles_cap);
  L->master = cv.take(4 * L->d_pad);
  L->ring = cv.take(L->esz * L->d_pad * (S + 1));
  L->G = cv.take(4 * L->d_pad * (lsq ? W : L->P));
  if (!lsq) {
    const int C = m->dims[m->n_layers];
    L->logits = cv.take(4 * (size_t)L->rows_cap * C);
    for (int l = 1; l <= m->n_layers; ++l) {
      L->act[l] = (l < m->n_layers) ? cv.take(L->esz * (size_t)L->rows_cap * m->dims[l]) : 0;
      L->delta[l] = cv.take(L->esz * (size_t)L->rows_cap * m->dims[l]);
    }
  }
  const size_t R = (size_t)m->max_rounds;
  L->tr_K = cv.take(4 * R);
  L->tr_R = cv.take(4 * R);
  L->tr_theta = cv.take(4 * R);
  L->tr_T = cv.take(8 * R);
  L->tr_loss = cv.take(4 * R);
  L->tr_comm = cv.take(8 * R);
  L->tr_sel_off = cv.take(8 * (R + 1));
  L->tr_rst_off = cv.take(8 * (R + 1));
  L->tr_sel_id = cv.take(4 * R * W);
  L->tr_sel_tau = cv.take(4 * R * W);
  L->tr_sel_loss = cv.take(4 * R * W);
  L->tr_rst_id = cv.take(4 * R * W);
  if (m->data_on_host) {
    L->data_X = cv.take(L->esz * (size_t)m->n_samples * m->dims[0]);
    L->data_y = cv.take(4 * (size_t)m->n_samples);
  }
  L->total = cv.off;
}

}  // namespace

struct abs_ctx {
  abs_model_desc m;
  Layout L;
  int W, K0, S;
  cudaStream_t stream;
  char* ws;
  const void* X;
  const void* y;
  int rounds_enqueued = 0;
  int sticky = ABS_OK;
  long long launches = 0;
  CtlArgs ctl;
  template <typename U> U* at(size_t off) const { return reinterpret_cast<U*>(ws + off); }
};

namespace {

int cuda_fail(abs_ctx* ctx, cudaError_t e, const char* what) {
  if (ctx) ctx->sticky = ABS_ECUDA;
  return fail(ABS_ECUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define CU(call)                                                   \
  do {                                                             \
    cudaError_t e_ = (call);                                       \
    if (e_ != cudaSuccess) return cuda_fail(ctx, e_, #call);       \
  } while (0)

template <typename T>
void enqueue_gradient(abs_ctx* ctx) {
  const abs_model_desc& m = ctx->m;
  const Layout& L = ctx->L;
  cudaStream_t s = ctx->stream;
  DevState* st = ctx->at<DevState>(L.st);
  if (m.kind == ABS_LSQ) {
    LsqArgs a;
    a.st = st; a.sel_tau = ctx->ctl.sel_tau; a.sel_row0 = ctx->ctl.sel_row0; a.row_idx = ctx->ctl.row_idx;
    a.X = ctx->X; a.y = (const float*)ctx->y;
    a.ring = ctx->at<void>(L.ring); a.slot_stride = L.d_pad;
    a.loss = ctx->ctl.loss; a.G = ctx->at<float>(L.G); a.d = m.dims[0];
    lsq_grad_kernel<T><<<ctx->W, 256, 0, s>>>(a);
    ctx->launches += 1;
    return;
  }
  const int nl = m.n_layers;
  const int row_tiles = L.rows_cap / TM;
  LayerArgs la[ABS_MAX_LAYERS];
  for (int l = 0; l < nl; ++l) {
    LayerArgs& a = la[l];
    a.st = st; a.tile_slot = ctx->ctl.tile_slot; a.row_idx = ctx->ctl.row_idx;
    a.ring = ctx->at<void>(L.ring); a.slot_stride = L.d_pad; a.w_off = L.w_off[l];
    a.in = m.dims[l]; a.out = m.dims[l + 1];
    a.gather = (l == 0);
    a.act_in = (l == 0) ? ctx->X : ctx->at<void>(L.act[l]);
    a.act_out = (l == nl - 1) ? ctx->at<void>(L.logits) : ctx->at<void>(L.act[l + 1]);
    a.delta_out = ctx->at<void>(L.delta[l + 1]);
    a.delta_in = (l == 0) ? nullptr : ctx->at<void>(L.delta[l]);
    a.G = ctx->at<float>(L.G); a.P = L.P;
  }
  for (int l = 0; l < nl; ++l) {
    dim3 grid((la[l].out + TN - 1) / TN, row_tiles);
    if (l == nl - 1) simt_fwd_kernel<T, true><<<grid, 256, 0, s>>>(la[l]);
    else simt_fwd_kernel<T, false><<<grid, 256, 0, s>>>(la[l]);
  }
  LossArgs lo;
  lo.st = st; lo.row_idx = ctx->ctl.row_idx; lo.labels = (const int*)ctx->y;
  lo.logits = ctx->at<float>(L.logits); lo.delta = ctx->at<void>(L.delta[nl]);
  lo.row_loss = ctx->ctl.row_loss; lo.C = m.dims[nl];
  net_loss_kernel<T><<<(L.rows_cap + 255) / 256, 256, 0, s>>>(lo);
  for (int l = nl - 1; l >= 0; --l) {
    if (l > 0) {
      dim3 grid((la[l].in + TN - 1) / TN, row_tiles);
      simt_dgrad_kernel<T><<<grid, 256, 0, s>>>(la[l]);
    }
    dim3 gridw((la[l].out + TN - 1) / TN, (la[l].in + 1 + TM - 1) / TM, L.P);
    simt_wgrad_kernel<T><<<gridw, 256, 0, s>>>(la[l]);
  }
  ctx->launches += 3 * nl;
}

template <typename T>
void enqueue_update(abs_ctx* ctx) {
  const Layout& L = ctx->L;
  UpdateArgs u;
  u.st = ctx->at<DevState>(L.st); u.master = ctx->at<float>(L.master); u.ring = ctx->at<void>(L.ring);
  u.G = ctx->at<float>(L.G); u.d_pad = L.d_pad; u.P = L.P; u.lr = ctx->m.lr;
  const size_t n4 = L.d_pad / 4;
  const int blocks = (int)std::min<size_t>((n4 + 255) / 256, 148 * 8);
  update_kernel<T><<<blocks, 256, 0, ctx->stream>>>(u);
  ctx->launches += 1;
}

int read_status(abs_ctx* ctx, DevState* host) {
  CU(cudaMemcpyAsync(host, ctx->at<DevState>(ctx->L.st), sizeof(DevState), cudaMemcpyDeviceToHost, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  return ABS_OK;
}

int status_to_code(abs_ctx* ctx, const DevState& h) {
  switch (h.status) {
    case ST_OK: return ABS_OK;
    case ST_DIVERGED:
      ctx->sticky = ABS_EDIVERGED;
      return fail(ABS_EDIVERGED, "non-finite loss uploaded in round %d; state is that of %d completed rounds", h.t, h.t);
    case ST_RANGE: ctx->sticky = ABS_ERANGE; return fail(ABS_ERANGE, "simulated time left the 2^53 tick range in round %d", h.t);
    case ST_NOSPACE: ctx->sticky = ABS_ENOSPACE; return fail(ABS_ENOSPACE, "round capacity %d exhausted", h.max_rounds);
    case ST_TIMEOUT: ctx->sticky = ABS_ETIMEOUT; return fail(ABS_ETIMEOUT, "bounded device wait expired (site %d)", h.timeout_where);
    default: ctx->sticky = ABS_ECUDA; return fail(ABS_ECUDA, "internal invariant failed (status %d, round %d)", h.status, h.t);
  }
}

}  // namespace

extern "C" {

const char* abs_last_error(void) { return g_err.c_str(); }

int abs_workspace_bytes(const abs_model_desc* model, int W, int staleness_bound, size_t* out) {
  if (!out) return fail(ABS_EINVAL, "out is null");
  const int rc = check_model(model, W, staleness_bound);
  if (rc != ABS_OK) return rc;
  Layout L;
  make_layout(model, W, staleness_bound, &L);
  *out = L.total;
  return ABS_OK;
}

int abs_init(abs_ctx** out, const abs_model_desc* model, int W, int K0, int staleness_bound,
             const abs_time_dist* td, unsigned long long seed) {
  abs_ctx* ctx = nullptr;
  if (!out) return fail(ABS_EINVAL, "out is null");
  *out = nullptr;
  int rc = check_model(model, W, staleness_bound);
  if (rc != ABS_OK) return rc;
  if (model->local_steps != 1)
    return fail(ABS_EUNSUPPORTED, "local_steps = %d: only U = 1 is implemented", model->local_steps);
  if (K0 < 1 || K0 > W) return fail(ABS_EINVAL, "K0 %d outside [1, W]", K0);
  if (model->k_mode != ABS_K_ADAPTIVE && model->k_mode != ABS_K_FIXED) return fail(ABS_EINVAL, "k_mode");
  if (model->bound_mode != ABS_BOUND_ADAPTIVE && model->bound_mode != ABS_BOUND_FIXED)
    return fail(ABS_EINVAL, "bound_mode");
  if (!(model->lr >= 0.f) || !std::isfinite(model->lr)) return fail(ABS_EINVAL, "lr");
  if (!td) return fail(ABS_EINVAL, "time_dist is null");
  if (td->kind < ABS_T_CONST || td->kind > ABS_T_PARETO2) return fail(ABS_EUNSUPPORTED, "time_dist kind %d", td->kind);
  if ((td->kind == ABS_T_EXP || td->kind == ABS_T_SHIFTED_EXP) && !(td->rate > 0.0)) return fail(ABS_EINVAL, "rate must be > 0");
  if ((td->kind == ABS_T_CONST || td->kind == ABS_T_SHIFTED_EXP) && !(td->shift >= 0.0)) return fail(ABS_EINVAL, "shift must be >= 0");
  if (td->kind == ABS_T_PARETO2 && !(td->scale > 0.0)) return fail(ABS_EINVAL, "scale must be > 0");
  if (td->slow_mod < 0 || (td->slow_mod > 0 && (td->slow_rem < 0 || td->slow_rem >= td->slow_mod)))
    return fail(ABS_EINVAL, "slow class");
  if (td->slow_mod > 0 && !(td->slow_factor > 0.0)) return fail(ABS_EINVAL, "slow_factor must be > 0");
  if (!model->X || !model->y || !model->w0) return fail(ABS_EINVAL, "X, y and w0 must be non-null");
  if (!model->workspace) return fail(ABS_EINVAL, "workspace is null");
  if (((uintptr_t)model->workspace & 255) != 0) return fail(ABS_EINVAL, "workspace must be 256-byte aligned");
  if (!model->data_on_host && (((uintptr_t)model->X & 15) != 0 || ((uintptr_t)model->y & 3) != 0))
    return fail(ABS_EINVAL, "X must be 16-byte aligned, y 4-byte aligned");
  Layout L;
  make_layout(model, W, staleness_bound, &L);
  if (model->workspace_bytes < L.total)
    return fail(ABS_ENOSPACE, "workspace has %zu bytes, %zu needed", model->workspace_bytes, L.total);

  ctx = new (std::nothrow) abs_ctx();
  if (!ctx) return fail(ABS_EINVAL, "out of host memory");
  ctx->m = *model; ctx->L = L; ctx->W = W; ctx->K0 = K0; ctx->S = staleness_bound;
  ctx->stream = (cudaStream_t)model->stream;
  ctx->ws = (char*)model->workspace;
  cudaStream_t s = ctx->stream;
  auto bail = [&](int code) { delete ctx; return code; };

  // everything except the dataset copy starts from zero (gradient padding must stay zero)
  const size_t zero_bytes = model->data_on_host ? L.data_X : L.total;
  cudaError_t e = cudaMemsetAsync(ctx->ws, 0, zero_bytes, s);
  if (e != cudaSuccess) return bail(cuda_fail(nullptr, e, "cudaMemsetAsync(workspace)"));
  if (model->data_on_host) {
    e = cudaMemcpyAsync(ctx->ws + L.data_X, model->X, L.esz * (size_t)model->n_samples * model->dims[0], cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->ws + L.data_y, model->y, 4 * (size_t)model->n_samples, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return bail(cuda_fail(nullptr, e, "dataset copy"));
    ctx->X = ctx->ws + L.data_X;
    ctx->y = ctx->ws + L.data_y;
  } else {
    ctx->X = model->X;
    ctx->y = model->y;
  }
  // w0 into the padded master layout
  for (int l = 0; l < model->n_layers; ++l) {
    const size_t n = model->kind == ABS_LSQ ? (size_t)model->dims[0]
                                             : (size_t)model->dims[l] * model->dims[l + 1] + model->dims[l + 1];
    e = cudaMemcpyAsync(ctx->at<float>(L.master) + L.w_off[l], model->w0 + L.w_src[l], 4 * n, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return bail(cuda_fail(nullptr, e, "w0 copy"));
  }
  DevState h;
  memset(&h, 0, sizeof h);
  h.W = W; h.K0 = K0; h.S = staleness_bound; h.B = model->batch; h.RB = L.RB;
  h.k_mode = model->k_mode; h.bound_mode = model->bound_mode; h.max_rounds = model->max_rounds;
  h.n_samples = model->n_samples;
  h.key0 = (uint32_t)(seed & 0xffffffffull); h.key1 = (uint32_t)(seed >> 32);
  h.dist.kind = td->kind; h.dist.shift = td->shift; h.dist.rate = td->rate; h.dist.scale = td->scale;
  h.dist.slow_mod = td->slow_mod; h.dist.slow_rem = td->slow_rem; h.dist.slow_factor = td->slow_factor;
  h.K = K0; h.theta = staleness_bound; h.comm = (u64)W;
  e = cudaMemcpyAsync(ctx->at<DevState>(L.st), &h, sizeof h, cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return bail(cuda_fail(nullptr, e, "state copy"));

  CtlArgs& c = ctx->ctl;
  c.st = ctx->at<DevState>(L.st);
  c.c = ctx->at<u64>(L.c); c.version = ctx->at<int>(L.version); c.job = ctx->at<int>(L.job);
  c.sel = ctx->at<int>(L.sel); c.sel_tau = ctx->at<int>(L.sel_tau); c.sel_row0 = ctx->at<int>(L.sel_row0);
  c.loss = ctx->at<float>(L.loss);
  c.row_loss = model->kind == ABS_LSQ ? nullptr : ctx->at<float>(L.row_loss);
  c.row_idx = ctx->at<int>(L.row_idx); c.tile_slot = ctx->at<int>(L.tile_slot);
  c.tr_K = ctx->at<int>(L.tr_K); c.tr_R = ctx->at<int>(L.tr_R); c.tr_theta = ctx->at<int>(L.tr_theta);
  c.tr_T = ctx->at<u64>(L.tr_T); c.tr_loss = ctx->at<float>(L.tr_loss); c.tr_comm = ctx->at<u64>(L.tr_comm);
  c.tr_sel_off = ctx->at<i64>(L.tr_sel_off); c.tr_rst_off = ctx->at<i64>(L.tr_rst_off);
  c.tr_sel_id = ctx->at<int>(L.tr_sel_id); c.tr_sel_tau = ctx->at<int>(L.tr_sel_tau);
  c.tr_sel_loss = ctx->at<float>(L.tr_sel_loss); c.tr_rst_id = ctx->at<int>(L.tr_rst_id);

  abs_init_state_kernel<<<(W + 255) / 256, 256, 0, s>>>(c);
  if (model->dtype == ABS_FP32) ring_init_kernel<float><<<148, 256, 0, s>>>(ctx->at<float>(L.master), ctx->at<void>(L.ring), L.d_pad);
  else ring_init_kernel<__nv_bfloat16><<<148, 256, 0, s>>>(ctx->at<float>(L.master), ctx->at<void>(L.ring), L.d_pad);
  ctx->launches += 2;
  e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return bail(cuda_fail(nullptr, e, "set-up kernels"));
  DevState back;
  rc = read_status(ctx, &back);
  if (rc != ABS_OK) return bail(rc);
  if (back.status != ST_OK) return bail(fail(ABS_ERANGE, "initial job durations out of tick range"));
  *out = ctx;
  g_err.clear();
  return ABS_OK;
}

int abs_enqueue_rounds(abs_ctx* ctx, int n) {
  if (!ctx) return fail(ABS_EINVAL, "ctx is null");
  if (ctx->sticky != ABS_OK) return fail(ctx->sticky, "context is in a failed state (%d)", ctx->sticky);
  if (n < 0) return fail(ABS_EINVAL, "n < 0");
  if (ctx->rounds_enqueued + n > ctx->m.max_rounds)
    return fail(ABS_ENOSPACE, "%d rounds requested, %d of capacity %d already used", n, ctx->rounds_enqueued, ctx->m.max_rounds);
  const bool f32 = ctx->m.dtype == ABS_FP32;
  for (int r = 0; r < n; ++r) {
    // the control kernel completes the previous round (if any) and selects this round's arrivals
    abs_ctl_kernel<<<1, 1024, 0, ctx->stream>>>(ctx->ctl, 1, 1);
    ctx->launches += 1;
    if (f32) { enqueue_gradient<float>(ctx); enqueue_update<float>(ctx); }
    else { enqueue_gradient<__nv_bfloat16>(ctx); enqueue_update<__nv_bfloat16>(ctx); }
  }
  if (n > 0) {
    abs_ctl_kernel<<<1, 1024, 0, ctx->stream>>>(ctx->ctl, 1, 0);
    ctx->launches += 1;
  }
  CU(cudaGetLastError());
  ctx->rounds_enqueued += n;
  return ABS_OK;
}

int abs_rounds_done(abs_ctx* ctx, int* rounds) {
  if (!ctx || !rounds) return fail(ABS_EINVAL, "null argument");
  if (ctx->sticky == ABS_ECUDA) return fail(ABS_ECUDA, "context is in a failed state");
  DevState h;
  const int rc = read_status(ctx, &h);
  if (rc != ABS_OK) return rc;
  *rounds = h.t;
  return status_to_code(ctx, h);
}

int abs_run_rounds(abs_ctx* ctx, int n) {
  int rc = abs_enqueue_rounds(ctx, n);
  if (rc != ABS_OK) return rc;
  int done = 0;
  return abs_rounds_done(ctx, &done);
}

int abs_get_params(abs_ctx* ctx, float* dst, size_t cap, size_t* d_out) {
  if (!ctx || !dst) return fail(ABS_EINVAL, "null argument");
  if (ctx->sticky == ABS_ECUDA) return fail(ABS_ECUDA, "context is in a failed state");
  const Layout& L = ctx->L;
  if (d_out) *d_out = L.d;
  if (cap < L.d) return fail(ABS_ENOSPACE, "destination holds %zu floats, %zu needed", cap, L.d);
  for (int l = 0; l < ctx->m.n_layers; ++l) {
    const size_t n = ctx->m.kind == ABS_LSQ ? (size_t)ctx->m.dims[0]
                                             : (size_t)ctx->m.dims[l] * ctx->m.dims[l + 1] + ctx->m.dims[l + 1];
    CU(cudaMemcpyAsync(dst + L.w_src[l], ctx->at<float>(L.master) + L.w_off[l], 4 * n, cudaMemcpyDeviceToHost, ctx->stream));
  }
  CU(cudaStreamSynchronize(ctx->stream));
  return ABS_OK;
}

int abs_get_trace(abs_ctx* ctx, int first, int n, abs_trace* o) {
  if (!ctx || !o) return fail(ABS_EINVAL, "null argument");
  if (ctx->sticky == ABS_ECUDA) return fail(ABS_ECUDA, "context is in a failed state");
  DevState h;
  int rc = read_status(ctx, &h);
  if (rc != ABS_OK) return rc;
  if (first < 0 || n < 0 || first + n > h.t)
    return fail(ABS_EINVAL, "rounds [%d, %d) requested, %d completed", first, first + n, h.t);
  if (n == 0) return ABS_OK;
  const Layout& L = ctx->L;
  cudaStream_t s = ctx->stream;
  std::vector<i64> so(n + 1), ro(n + 1);
  CU(cudaMemcpyAsync(so.data(), ctx->at<i64>(L.tr_sel_off) + first, 8 * (size_t)(n + 1), cudaMemcpyDeviceToHost, s));
  CU(cudaMemcpyAsync(ro.data(), ctx->at<i64>(L.tr_rst_off) + first, 8 * (size_t)(n + 1), cudaMemcpyDeviceToHost, s));
  CU(cudaStreamSynchronize(s));
  const size_t n_sel = (size_t)(so[n] - so[0]), n_rst = (size_t)(ro[n] - ro[0]);
  if ((o->sel_id || o->sel_tau || o->sel_loss) && o->cap_sel < n_sel)
    return fail(ABS_ENOSPACE, "cap_sel %zu, %zu needed", o->cap_sel, n_sel);
  if (o->rst_id && o->cap_rst < n_rst) return fail(ABS_ENOSPACE, "cap_rst %zu, %zu needed", o->cap_rst, n_rst);
#define D2H(dst, off, type, start, count)                                                              \
  if ((dst) && (count) > 0)                                                                            \
    CU(cudaMemcpyAsync((dst), ctx->at<type>(off) + (start), sizeof(type) * (size_t)(count), cudaMemcpyDeviceToHost, s))
  D2H(o->K, L.tr_K, int, first, n);
  D2H(o->n_restart, L.tr_R, int, first, n);
  D2H(o->theta, L.tr_theta, int, first, n);
  D2H(o->T_end, L.tr_T, u64, first, n);
  D2H(o->loss_mean, L.tr_loss, float, first, n);
  D2H(o->comm, L.tr_comm, u64, first, n);
  D2H(o->sel_id, L.tr_sel_id, int, so[0], n_sel);
  D2H(o->sel_tau, L.tr_sel_tau, int, so[0], n_sel);
  D2H(o->sel_loss, L.tr_sel_loss, float, so[0], n_sel);
  D2H(o->rst_id, L.tr_rst_id, int, ro[0], n_rst);
#undef D2H
  CU(cudaStreamSynchronize(s));
  if (o->sel_off) for (int i = 0; i <= n; ++i) o->sel_off[i] = so[i] - so[0];
  if (o->rst_off) for (int i = 0; i <= n; ++i) o->rst_off[i] = ro[i] - ro[0];
  return ABS_OK;
}

int abs_launch_count(abs_ctx* ctx, long long* launches) {
  if (!ctx || !launches) return fail(ABS_EINVAL, "null argument");
  *launches = ctx->launches;
  return ABS_OK;
}

int abs_destroy(abs_ctx* ctx) {
  if (!ctx) return ABS_OK;
  cudaStreamSynchronize(ctx->stream);
  delete ctx;
  return ABS_OK;
}

}  // extern "C"
