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
#include "narrow.cuh"
#include "tc.cuh"
#include "outlayer.cuh"
#include "lsqpipe.cuh"
#include "local.cuh"
#include "localnet.cuh"
#include "persist.cuh"
#include "conv.cuh"

using namespace absb;

namespace {

thread_local std::string g_err;

}  // namespace

namespace absb {
void set_last_error(const char* text) { g_err = text; }
}

namespace {

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
enum LayerPath : int { PATH_SIMT = 0, PATH_TC = 1, PATH_NARROW = 2 };

struct Layout {
  int n_layers = 0, RB = 0, rows_cap = 0, P = 0, n_tiles_cap = 0;
  int path[ABS_MAX_LAYERS] = {};        // how each layer's contractions run
  int bn_fwd[ABS_MAX_LAYERS] = {}, bn_dg[ABS_MAX_LAYERS] = {}, bn_wg[ABS_MAX_LAYERS] = {};
  bool any_tc = false;
  int cg_fwd[ABS_MAX_LAYERS] = {}, cg_dg[ABS_MAX_LAYERS] = {}, cg_wg[ABS_MAX_LAYERS] = {};
  bool pair_bwd[ABS_MAX_LAYERS] = {};   // delta back-propagation and weight gradient of the layer share a launch
  bool bias_colsum[ABS_MAX_LAYERS] = {}; // the layer's bias gradient = column sums of the delta the layer above back-propagates
  size_t colsum[ABS_MAX_LAYERS] = {};   // [rows_cap / 32][out] those sums per group of 32 rows
  int fused_R = 0;                      // rows per block of the fused output-layer kernel (0: not used)
  int narrow_rpb = 64;                  // rows per block of the row-tiled output-layer kernels that are not fused
  bool out_mma = false;                 // output layer through the mma.sync kernel (bf16, 64 rows per CTA)
  size_t esz = 4;                       // bytes per stored element (4 or 2)
  size_t d = 0, d_pad = 0;
  size_t w_off[ABS_MAX_LAYERS] = {};    // element offset of W_l inside the padded vector
  size_t w_src[ABS_MAX_LAYERS] = {};    // element offset of W_l inside the caller's vector
  size_t st, ri, c, version, job, next_dur, dur_job, loss, row_loss;
  size_t sel[2], sel_tau[2], sel_row0[2], row_idx[2], tile_slot[2];   // per-round layout, by round parity
  size_t act0b;                         // second copy of the gathered input rows (odd rounds)
  size_t master, ring, G, logits, red, ones;
  // convolution blocks of ABS_CNN (two of them, in front of the affine layers)
  bool cnn = false;
  int cHi[2] = {}, cWi[2] = {}, cCi[2] = {}, cCo[2] = {}, ck = 0;   // input map, channels of each block
  size_t c_off[2] = {}, c_src[2] = {}, c_len[2] = {};               // W[k][k][Ci][Co] + b[Co]: padded / caller offset, length
  size_t x_len = 0;                       // elements of one dataset row
  size_t pool1 = 0, dpool1 = 0, arg1 = 0, arg2 = 0, cpart[2] = {};  // pooled maps of block 1, their delta, pool positions, chunk sums
  int cchunk = 1;                         // gradient rows per CTA of the convolution weight-gradient kernel
  size_t bits[ABS_MAX_LAYERS + 1];      // ReLU sign bits of act[l] (tensor-core layers)
  size_t act[ABS_MAX_LAYERS + 1], delta[ABS_MAX_LAYERS + 1];
  size_t tr_K, tr_R, tr_theta, tr_T, tr_loss, tr_comm, tr_sel_off, tr_rst_off;
  size_t tr_sel_id, tr_sel_tau, tr_sel_loss, tr_rst_id;
  size_t data_X, data_y;
  // U > 1 on a multi-layer network: the selected workers' own model copies and uploads
  bool local_net = false;
  int RBp = 0;                          // rows reserved per worker in a local step's row layout
  size_t priv = 0, loss_acc = 0;          // the workers' copies (storage type); their uploads live in G
  size_t gring = 0;                     // the models the gradient kernels read: the ring, or the private copies
  int gslots = 0;
  size_t total = 0;
};

int check_model(const abs_model_desc* m, int W, int S) {
  if (!m) return fail(ABS_EINVAL, "model is null");
  if (m->kind != ABS_LSQ && m->kind != ABS_SOFTMAX && m->kind != ABS_MLP && m->kind != ABS_CNN)
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
  if (m->kind == ABS_CNN) {
    const int H = m->conv[0], Wd = m->conv[1], Ci = m->conv[2], k = m->conv[3], C1 = m->conv[4], C2 = m->conv[5];
    if (m->n_layers < 2) return fail(ABS_EINVAL, "ABS_CNN needs at least two affine layers behind the convolution blocks");
    if (H < 1 || Wd < 1 || Ci < 1 || k < 1 || C1 < 1 || C2 < 1 || H > 1024 || Wd > 1024 || Ci > 1024 || C1 > 1024 || C2 > 1024)
      return fail(ABS_EINVAL, "conv = {H, W, C_in, k, C1, C2} out of range");
    const int H1 = H - k + 1, W1 = Wd - k + 1;
    if (H1 < 2 || W1 < 2 || (H1 & 1) || (W1 & 1)) return fail(ABS_EINVAL, "first convolution output %d x %d must be even-sized and at least 2 x 2", H1, W1);
    const int H2 = H1 / 2 - k + 1, W2 = W1 / 2 - k + 1;
    if (H2 < 2 || W2 < 2 || (H2 & 1) || (W2 & 1)) return fail(ABS_EINVAL, "second convolution output %d x %d must be even-sized and at least 2 x 2", H2, W2);
    if ((long long)(H2 / 2) * (W2 / 2) * C2 != m->dims[0])
      return fail(ABS_EINVAL, "dims[0] = %d, but the second block delivers %d features", m->dims[0], (H2 / 2) * (W2 / 2) * C2);
    if ((long long)k * k * Ci * C1 + C1 > 4096 || (long long)k * k * C1 * C2 + C2 > 4096)
      return fail(ABS_EUNSUPPORTED, "a convolution block may have at most 4096 parameters");
    if (conv::bwd_smem_bytes(H, Wd, Ci, k, C1) > 200 * 1024 || conv::bwd_smem_bytes(H1 / 2, W1 / 2, C1, k, C2) > 200 * 1024)
      return fail(ABS_EUNSUPPORTED, "convolution maps too large for the shared-memory kernels");
    if (m->local_steps > 1) return fail(ABS_EUNSUPPORTED, "local_steps > 1 is not implemented for ABS_CNN");
  }
  if (m->batch < 1 || m->batch > 1024) return fail(ABS_EINVAL, "batch %d outside [1, 1024]", m->batch);
  if (m->max_rounds < 1) return fail(ABS_EINVAL, "max_rounds %d < 1", m->max_rounds);
  if (m->n_samples < 1 || m->n_samples > 0x7fffffffLL) return fail(ABS_EINVAL, "n_samples out of range");
  if (W < 1 || W > ABS_MAX_WORKERS) return fail(ABS_EINVAL, "W %d outside [1, %d]", W, ABS_MAX_WORKERS);
  if (m->n_samples < W) return fail(ABS_EINVAL, "fewer samples than workers");
  if (S < 0 || S > ABS_MAX_BOUND) return fail(ABS_EINVAL, "staleness_bound %d outside [0, %d]", S, ABS_MAX_BOUND);
  if (m->restart_rule != ABS_RESTART_ALGORITHM1 && m->restart_rule != ABS_RESTART_EQ6 && m->restart_rule != ABS_RESTART_NONE)
    return fail(ABS_EINVAL, "restart_rule");
  if (m->sa_penalty != 0 && m->sa_penalty != 1) return fail(ABS_EINVAL, "sa_penalty must be 0 or 1");
  if (m->restart_rule == ABS_RESTART_EQ6 && S + 1 > ABS_MAX_BOUND)
    return fail(ABS_EINVAL, "staleness_bound %d: Eq. 6 as printed keeps one more version, at most %d", S, ABS_MAX_BOUND - 1);
  return ABS_OK;
}

void make_layout(const abs_model_desc* m, int W, int S, Layout* L) {
  L->n_layers = m->n_layers;
  L->esz = m->dtype == ABS_FP32 ? 4 : 2;
  const bool lsq = m->kind == ABS_LSQ;
  // padded parameter vector: each layer's [W | b] block starts on a 64-element boundary
  size_t off = 0, src = 0;
  L->cnn = m->kind == ABS_CNN;
  L->x_len = (size_t)m->dims[0];
  if (L->cnn) {
    const int H = m->conv[0], Wd = m->conv[1], k = m->conv[3];
    L->ck = k;
    L->cHi[0] = H; L->cWi[0] = Wd; L->cCi[0] = m->conv[2]; L->cCo[0] = m->conv[4];
    L->cHi[1] = (H - k + 1) / 2; L->cWi[1] = (Wd - k + 1) / 2; L->cCi[1] = m->conv[4]; L->cCo[1] = m->conv[5];
    L->x_len = (size_t)H * Wd * m->conv[2];
    for (int b = 0; b < 2; ++b) {
      L->c_len[b] = (size_t)k * k * L->cCi[b] * L->cCo[b] + L->cCo[b];
      L->c_off[b] = off; L->c_src[b] = src;
      off = round_up_sz(off + L->c_len[b], 64);
      src += L->c_len[b];
    }
  }
  for (int l = 0; l < m->n_layers; ++l) {
    L->w_off[l] = off;
    L->w_src[l] = src;
    const size_t n = lsq ? (size_t)m->dims[0] : (size_t)m->dims[l] * m->dims[l + 1] + m->dims[l + 1];
    off = round_up_sz(off + n, 64);
    src += n;
  }
  L->d = src;
  L->d_pad = round_up_sz(off, 256);
  // per-layer path: tensor cores for bf16 hidden layers whose sizes TMA can address, the
  // narrow-output kernels for a last layer of at most 16 classes, FP32-FMA tiles otherwise
  const bool tc_ok = m->dtype == ABS_BF16_FP32MASTER && !(m->flags & ABS_FLAG_NO_TENSOR_CORES);
  L->any_tc = false;
  for (int l = 0; l < m->n_layers && !lsq; ++l) {
    const int in = m->dims[l], out = m->dims[l + 1];
    const bool last = l == m->n_layers - 1;
    if (last && out <= NARROW_MAX_C && (size_t)in * out <= 10240) L->path[l] = PATH_NARROW;
    else if (!last && tc_ok && in % 8 == 0 && out % 8 == 0 && in >= 64 && out >= 64) {
      L->path[l] = PATH_TC;
      L->any_tc = true;
    } else L->path[l] = PATH_SIMT;
  }
  L->RB = lsq ? m->batch : (L->any_tc ? 128 : 64);
  const int groups = (W < S + 1) ? W : S + 1;
  L->rows_cap = round_up(W * m->batch, L->RB) + groups * L->RB;
  L->local_net = !lsq && m->n_layers > 1 && m->local_steps > 1;
  if (L->local_net) {
    L->RBp = round_up(m->batch, L->RB);
    L->rows_cap = std::max(L->rows_cap, W * L->RBp);
  }
  L->n_tiles_cap = L->rows_cap / L->RB;
  if (lsq) {
    L->P = 0;
  } else if (L->any_tc) {
    // tile widths: widest tile that still gives every SM work; split count of the row reduction
    // sized so the largest weight gradient fills about two waves of 148 CTAs
    const int row_tiles = L->rows_cap / 128;
    auto pick = [](int n, int other_tiles) {
      for (int bn : {256, 128}) if (n >= bn && other_tiles * ((n + bn - 1) / bn) >= 120) return bn;
      return n >= 128 ? 128 : 64;
    };
    for (int l = 0; l < m->n_layers; ++l) {
      if (L->path[l] != PATH_TC) continue;
      const int in = m->dims[l], out = m->dims[l + 1];
      L->bn_fwd[l] = pick(out, row_tiles);
      L->bn_dg[l] = pick(in, row_tiles);
      L->bn_wg[l] = pick(out, ((in + 127) / 128 + 1) * 3);
      L->cg_fwd[l] = L->cg_dg[l] = L->cg_wg[l] = 1;
      if ((size_t)in * out >= ((size_t)1 << 21) && in >= 256 && out >= 256 && W * m->batch >= 4096) {
        // a large weight gradient is bound by operand traffic into shared memory: CTA pairs halve
        // the B operand each CTA has to stage (its tiles are features x outputs, so the row padding
        // unit of the version groups is not involved)
        L->cg_wg[l] = 2; L->bn_wg[l] = 256;
      }
    }
    // A short weight gradient (fewer tiles than SMs at the back-propagation's tile width) shares
    // its launch with the layer's delta back-propagation: both have one or two tiles per CTA, so
    // separate launches would pay the fixed costs of a launch twice.
    for (int l = 1; l < m->n_layers; ++l) {
      if (L->path[l] != PATH_TC || L->cg_dg[l] != 1 || L->cg_wg[l] != 1 || (m->flags & ABS_FLAG_NO_FUSED_BACKWARD)) continue;
      if (L->local_net) continue;
      const int in = m->dims[l], out = m->dims[l + 1], bn = L->bn_dg[l];
      if (out < bn) continue;
      const long wg_tiles_min = (long)((in + 127) / 128 + 1) * ((out + bn - 1) / bn);   // at P = 1
      if (wg_tiles_min * 4 < 148) { L->pair_bwd[l] = true; L->bn_wg[l] = bn; }
    }
    // A layer whose output delta is produced by the tensor-core back-propagation of the layer above gets its bias
    // gradient from column sums taken in that kernel's epilogue; its weight gradient then needs no row tile of ones.
    // (for at most as many layers as the Eq. 3 kernel takes partial-sum regions besides the output layer's)
    for (int l = 0, n = 0; l + 1 < m->n_layers; ++l) {
      L->bias_colsum[l] = L->path[l] == PATH_TC && L->path[l + 1] == PATH_TC && !L->local_net && m->local_steps <= 1 &&
                          n < UpdateArgs::MAX_REGIONS - 1;
      n += L->bias_colsum[l] ? 1 : 0;
    }
    // split count P of the row reduction: the one that minimises the modelled time of all weight
    // gradients (whole waves of 148 CTAs, one tile = 128 x BN x rows/P) plus the extra partial
    // sums the Eq. 3 step then has to read
    double best = 1e30;
    int bestP = 1;
    // splits of at least 512 rows, at most 4: each split is one more partial vector for the Eq. 3 step (7 splits cost
    // it 12 us on configuration 4 and win the weight gradient nothing), and on small models a weight gradient spread
    // over more CTAs takes the SMs the side-stream kernels of the next round run on (configuration 3: 8 splits make
    // the kernel 4 us shorter and the round 5 us longer)
    // (the CNN's affine layers see at most a few hundred rows per round and run on one stream: splits of 128 rows,
    // so that its FP32 weight-gradient kernels, whose grid is tiles x splits, are more than a handful of CTAs)
    const int maxP = std::max(1, std::min(4, W * m->batch / (L->cnn ? 128 : 512)));
    for (int P = 1; P <= maxP; ++P) {
      double t = 4.0 * (double)L->d_pad * P / 5e12;
      for (int l = 0; l < m->n_layers; ++l) {
        if (L->path[l] != PATH_TC) continue;
        const int in = m->dims[l], out = m->dims[l + 1], bn = L->bn_wg[l];
        const int cg = L->cg_wg[l], tm = 128 * cg, units = 148 / cg;
        const long tiles = (long)((in + tm - 1) / tm + (L->bias_colsum[l] ? 0 : 1)) * ((out + bn - 1) / bn) * P;
        const long waves = (tiles + units - 1) / units;
        t += (double)waves * 2.0 * 128.0 * bn * ((double)L->rows_cap / P) / 9e12;
      }
      if (t < best * 0.999) { best = t; bestP = P; }
    }
    L->P = bestP;
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
  L->ri = cv.take(2 * sizeof(RoundInfo));
  L->c = cv.take(sizeof(u64) * W);
  L->version = cv.take(4 * W);
  L->job = cv.take(4 * W);
  L->next_dur = cv.take(8 * W);
  L->dur_job = cv.take(4 * W);
  for (int q = 0; q < 2; ++q) {
    L->sel[q] = cv.take(4 * W);
    L->sel_tau[q] = cv.take(4 * W);
    L->sel_row0[q] = cv.take(4 * W);
    L->row_idx[q] = cv.take(4 * (size_t)L->rows_cap);
    L->tile_slot[q] = cv.take(4 * (size_t)L->n_tiles_cap);
  }
  L->loss = cv.take(4 * W);
  L->row_loss = cv.take(4 * (size_t)L->rows_cap);
  L->master = cv.take(4 * L->d_pad);
  L->ring = cv.take(L->esz * L->d_pad * (S + 1));
  if (m->local_steps > 1) L->P = 0;      // Eq. 3 adds one upload per selected worker
  L->G = cv.take(4 * L->d_pad * ((lsq || m->local_steps > 1) ? W : L->P));
  L->gring = L->ring;
  L->gslots = S + 1;
  if (L->local_net) {
    L->priv = cv.take(L->esz * L->d_pad * W);
    L->loss_acc = cv.take(4 * W);
    L->gring = L->priv;
    L->gslots = W;
  }
  if (!lsq) {
    const int C = m->dims[m->n_layers];
    L->logits = cv.take(4 * (size_t)L->rows_cap * C);
    {
      // chunk partials of the two-stage column reductions (bias sums, output-layer gradient)
      size_t len = (size_t)(m->dims[m->n_layers - 1] + 1) * C;
      for (int l = 0; l < m->n_layers; ++l) len = std::max(len, (size_t)m->dims[l + 1]);
      // the fused output-layer kernel keeps R input rows in shared memory
      const int inl = m->dims[m->n_layers - 1];
      L->fused_R = 0;
      if (L->path[m->n_layers - 1] == PATH_NARROW && inl % 8 == 0)
        for (int R : {32, 16, 8})     // (rows, transposed weights in fp32 or storage type, stored weights, deltas)
          if ((size_t)R * inl * L->esz + (size_t)C * (inl + 8) * 4 + (size_t)(inl + 1) * C * L->esz + 64 +
                  (size_t)R * 64 <= 100 * 1024) { L->fused_R = R; break; }
      L->out_mma = L->fused_R && tc_ok && m->n_layers > 1 &&
                   (inl == 128 || inl == 256 || inl == 512 || inl == 1024);
      // the non-fused output-layer kernels: fewer rows per block when a round has few rows, so that the grid is
      // more than a handful of blocks (each is a chain of dependent loads)
      L->narrow_rpb = 64;
      if (!L->local_net)
        while (L->narrow_rpb > 8 && (long long)W * m->batch / L->narrow_rpb < 2 * 148) L->narrow_rpb /= 2;
      L->red = cv.take(4 * len * (size_t)(L->rows_cap / (L->fused_R ? L->fused_R : L->narrow_rpb)));
    }
    L->ones = L->any_tc ? cv.take(2 * 64 * (size_t)L->rows_cap) : 0;
    for (int l = 0; l < m->n_layers; ++l)
      if (L->bias_colsum[l]) L->colsum[l] = cv.take(4 * (size_t)(L->rows_cap / 32) * m->dims[l + 1]);
    for (int l = 0; l <= m->n_layers; ++l) L->bits[l] = 0;
    for (int l = 0; l + 1 < m->n_layers; ++l)
      if (L->path[l] == PATH_TC) L->bits[l + 1] = cv.take(4 * (size_t)L->rows_cap * ((m->dims[l + 1] + 31) / 32));
    const bool copy0 = L->path[0] == PATH_TC || L->cnn;     // gathered copies of the input rows (CNN: the features)
    L->act[0] = copy0 ? cv.take(L->esz * (size_t)L->rows_cap * m->dims[0]) : 0;
    L->act0b = copy0 ? cv.take(L->esz * (size_t)L->rows_cap * m->dims[0]) : 0;
    for (int l = 1; l <= m->n_layers; ++l) {
      L->act[l] = (l < m->n_layers) ? cv.take(L->esz * (size_t)L->rows_cap * m->dims[l]) : 0;
      L->delta[l] = cv.take(L->esz * (size_t)L->rows_cap * m->dims[l]);
    }
    if (L->cnn) {
      const size_t n_p1 = (size_t)L->cHi[1] * L->cWi[1] * L->cCi[1];        // pooled maps of block 1 per row
      L->delta[0] = cv.take(L->esz * (size_t)L->rows_cap * m->dims[0]);
      L->pool1 = cv.take(L->esz * (size_t)L->rows_cap * n_p1);
      L->dpool1 = cv.take(L->esz * (size_t)L->rows_cap * n_p1);
      L->arg1 = cv.take((size_t)L->rows_cap * n_p1);
      L->arg2 = cv.take((size_t)L->rows_cap * m->dims[0]);
      // rows per weight-gradient CTA: the largest power of two that still leaves four CTAs per SM when every
      // worker is selected (a CTA is 8 warps on a chain of shared-memory loads: measured on 640 rows per round,
      // 1 / 2 / 4 / 8 rows per CTA give 1742 / 1617 / 1409 / 1222 rounds/s)
      L->cchunk = 1;
      while (L->cchunk < conv::MAX_CHUNK && (long long)W * m->batch / (2 * L->cchunk) >= 4 * 148) L->cchunk *= 2;
      for (int b = 0; b < 2; ++b) L->cpart[b] = cv.take(4 * L->c_len[b] * (size_t)(L->rows_cap / L->cchunk));
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
    L->data_X = cv.take(L->esz * (size_t)m->n_samples * L->x_len);
    L->data_y = cv.take(4 * (size_t)m->n_samples);
  }
  L->total = cv.off;
}

}  // namespace

struct TcLayer {
  CUtensorMap fwd_a, fwd_b, dg_a, dg_b, wg_a, wg_b;
  CUtensorMap fwd_out, dg_out, wg_out;     // result tensors written by bulk tensor stores
  CUtensorMap fwd_a_odd, wg_a_odd;         // layer 0 only: operand maps over the second gathered copy
};

// ones[r][0] = 1 (bf16), the rest of the 64-wide rows stays zero: the extra operand row that turns
// the weight-gradient GEMM into weight + bias gradient
__global__ void ones_init_kernel(__nv_bfloat16* ones, int rows) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r < rows) ones[(size_t)r * 64] = __float2bfloat16_rn(1.f);
}

struct abs_ctx {
  abs_model_desc m;
  Layout L;
  int W, K0, S;
  int sm_count = 148;
  cudaStream_t stream;
  // The control kernel (and the row gather) of round t+1 only need the losses of round t, so they
  // run on a second stream next to the backward kernels of round t.
  cudaStream_t side = nullptr;
  cudaEvent_t ev_loss = nullptr, ev_ctl = nullptr;
  bool overlap = false;
  char* ws;
  const void* X;
  const void* y;
  int rounds_enqueued = 0;
  int sticky = ABS_OK;
  long long launches = 0;
  cudaError_t launch_error = cudaSuccess;
  int next_cluster = 1;              // cluster width of the next launch (consumed by launch_on)
  int upd_blocks_per_sm = 8;         // resident blocks per SM of the Eq. 3 kernel
  bool local_sgd = false;            // U > 1: one CTA per selected worker runs the worker's local steps
  bool lsq_pipe = false;             // bf16 least squares through the bulk-copy pipeline kernel
  int lsq_stages = 0;
  bool lsq_v2 = false;               // least squares through the persistent 16-byte-load kernel
  int lsq_grid = 0;                  // its grid = number of partial sums
  bool lsq_rounds = false;           // small least squares: all enqueued rounds in one persistent kernel
  CtlArgs ctl;
  TcLayer tcl[ABS_MAX_LAYERS];
  CUtensorMap ones_map;
  // profiling: event pairs around launches
  std::vector<cudaEvent_t> ev;       // 2 per recorded launch
  std::vector<int> ev_class;
  int ev_cap = 0;                    // launches that may still be recorded
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

// One kernel launch on ctx->stream, counted and, while profiling, bracketed by events.  Launches
// carry the programmatic-stream-serialization attribute: the next kernel's CTAs may be scheduled
// while this one drains; every kernel of the round loop starts with griddepcontrol.wait, which
// returns once the kernel before it has completed and its writes are visible.
template <typename... KArgs, typename... Args>
void launch_on(abs_ctx* ctx, cudaStream_t stream, int cls, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
               Args&&... args) {
  const bool rec = (int)ctx->ev_class.size() < ctx->ev_cap;
  if (rec) cudaEventRecord(ctx->ev[2 * ctx->ev_class.size()], stream);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (ctx->next_cluster > 1) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)ctx->next_cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
    ctx->next_cluster = 1;
  }
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
  if (e != cudaSuccess && ctx->launch_error == cudaSuccess) ctx->launch_error = e;
  if (rec) {
    cudaEventRecord(ctx->ev[2 * ctx->ev_class.size() + 1], stream);
    ctx->ev_class.push_back(cls);
  }
  ctx->launches += 1;
}

template <typename... KArgs, typename... Args>
void launch_ex(abs_ctx* ctx, int cls, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, Args&&... args) {
  launch_on(ctx, ctx->stream, cls, kernel, grid, block, smem, static_cast<Args&&>(args)...);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// bf16 tensor map with 128-byte swizzle; dims/strides innermost first, strides in bytes for dims 1...
bool make_map(CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides,
              const cuuint32_t* box, CUtensorMapDataType dt = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, dt, (cuuint32_t)rank, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_act_map(CUtensorMap* map, const void* base, int dim, int rows, int box_rows) {
  const cuuint64_t dims[2] = {(cuuint64_t)dim, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)dim * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  return make_map(map, base, 2, dims, strides, box);
}

bool make_w_map(CUtensorMap* map, const void* base, int in, int out, int slots, size_t slot_stride, int box_rows) {
  const cuuint64_t dims[3] = {(cuuint64_t)out, (cuuint64_t)in, (cuuint64_t)slots};
  const cuuint64_t strides[2] = {(cuuint64_t)out * 2, (cuuint64_t)slot_stride * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  return make_map(map, base, 3, dims, strides, box);
}

// fp32 gradient block of one layer inside the partial-sum buffers: (out, in, P), 32 x 32 boxes
bool make_g_map(CUtensorMap* map, const void* base, int in, int out, int P, size_t slot_stride) {
  const cuuint64_t dims[3] = {(cuuint64_t)out, (cuuint64_t)in, (cuuint64_t)P};
  const cuuint64_t strides[2] = {(cuuint64_t)out * 4, (cuuint64_t)slot_stride * 4};
  const cuuint32_t box[3] = {32, 32, 1};
  return make_map(map, base, 3, dims, strides, box, CU_TENSOR_MAP_DATA_TYPE_FLOAT32);
}

// One problem (second = null), or two independent problems in one launch.
struct TcProblem { const CUtensorMap* a; const CUtensorMap* b; const CUtensorMap* o; const tc::Params* p; int max_tiles; };

template <int BN, int CG>
void launch_tc(abs_ctx* ctx, int cls, const TcProblem& x, const TcProblem* y) {
  const int units = ctx->sm_count / CG;           // CTAs, or CTA pairs
  const int grid = CG * std::max(1, std::min(units, x.max_tiles + (y ? y->max_tiles : 0)));
  tc::Params none;
  memset(&none, 0, sizeof none);
  none.mode = -1;
  ctx->next_cluster = CG;
  launch_ex(ctx, cls, tc::tc_gemm_kernel<BN, CG>, dim3(grid), dim3(tc::THREADS), tc::Cfg<BN, CG>::SMEM_BYTES, *x.a, *x.b,
            ctx->ones_map, *x.o, *x.p, *(y ? y->a : x.a), *(y ? y->b : x.b), *(y ? y->o : x.o), y ? *y->p : none);
}

// max_tiles counts tiles of (128 * cg) x bn
void launch_tc_bn(abs_ctx* ctx, int bn, int cg, int cls, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& o,
                  const tc::Params& p, int max_tiles, const TcProblem* second = nullptr) {
  const TcProblem x = {&a, &b, &o, &p, max_tiles};
  if (cg == 2) launch_tc<256, 2>(ctx, cls, x, second);
  else if (bn == 256) launch_tc<256, 1>(ctx, cls, x, second);
  else if (bn == 128) launch_tc<128, 1>(ctx, cls, x, second);
  else launch_tc<64, 1>(ctx, cls, x, second);
}

int setup_tc(abs_ctx* ctx) {
  const abs_model_desc& m = ctx->m;
  const Layout& L = ctx->L;
  if (!L.any_tc) return ABS_OK;
  cudaError_t e;
  e = cudaFuncSetAttribute(tc::tc_gemm_kernel<256, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::Cfg<256, 1>::SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc::tc_gemm_kernel<128, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::Cfg<128, 1>::SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc::tc_gemm_kernel<64, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::Cfg<64, 1>::SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc::tc_gemm_kernel<256, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::Cfg<256, 2>::SMEM_BYTES);
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaFuncSetAttribute(tc_gemm_kernel)");
  const char* ring = ctx->at<char>(L.gring);
  const int n_splits = L.P > 0 ? L.P : ctx->W;     // P = 0: one weight-gradient split per selected worker
  if (!make_act_map(&ctx->ones_map, ctx->at<void>(L.ones), 64, L.rows_cap, 64))
    return fail(ABS_ECUDA, "cuTensorMapEncodeTiled failed for the ones matrix");
  ones_init_kernel<<<(L.rows_cap + 255) / 256, 256, 0, ctx->stream>>>(ctx->at<__nv_bfloat16>(L.ones), L.rows_cap);
  ctx->launches += 1;
  for (int l = 0; l < m.n_layers; ++l) {
    if (L.path[l] != PATH_TC) continue;
    const int in = m.dims[l], out = m.dims[l + 1];
    TcLayer& t = ctx->tcl[l];
    const void* act_in = ctx->at<void>(L.act[l]);
    const void* delta_out = ctx->at<void>(L.delta[l + 1]);
    const void* wbase = ring + 2 * L.w_off[l];
    bool ok = make_act_map(&t.fwd_a, act_in, in, L.rows_cap, 128) &&
              make_w_map(&t.fwd_b, wbase, in, out, L.gslots, L.d_pad, 64) &&
              make_act_map(&t.wg_a, act_in, in, L.rows_cap, 64) &&
              make_act_map(&t.wg_b, delta_out, out, L.rows_cap, 64) &&
              make_act_map(&t.fwd_out, ctx->at<void>(L.act[l + 1]), out, L.rows_cap, 32) &&
              make_g_map(&t.wg_out, ctx->at<float>(L.G) + L.w_off[l], in, out, n_splits, L.d_pad);
    if (ok && l == 0)
      ok = make_act_map(&t.fwd_a_odd, ctx->at<void>(L.act0b), in, L.rows_cap, 128) &&
           make_act_map(&t.wg_a_odd, ctx->at<void>(L.act0b), in, L.rows_cap, 64);
    if (ok && (l > 0 || L.cnn))
      ok = make_act_map(&t.dg_a, delta_out, out, L.rows_cap, 128) &&
           make_w_map(&t.dg_b, wbase, in, out, L.gslots, L.d_pad, L.bn_dg[l] / L.cg_dg[l]) &&
           make_act_map(&t.dg_out, ctx->at<void>(L.delta[l]), in, L.rows_cap, 32);
    if (!ok) return fail(ABS_ECUDA, "cuTensorMapEncodeTiled failed for layer %d", l);
  }
  return ABS_OK;
}

enum Phase : int { PH_GATHER = 0, PH_FORWARD = 1, PH_BACKWARD = 2 };

// Kernels of one round, `par` = round parity (layout copy).  PH_GATHER: minibatch row copy (runs on
// the side stream when rounds overlap).  PH_FORWARD: everything up to the uploaded losses.
// PH_BACKWARD: the rest of the gradient.
template <typename T>
void enqueue_gradient(abs_ctx* ctx, int par, int phase) {
  const abs_model_desc& m = ctx->m;
  const Layout& L = ctx->L;
  cudaStream_t s = ctx->stream;
  DevState* st = ctx->at<DevState>(L.st);
  RoundInfo* ri = ctx->at<RoundInfo>(L.ri) + par;
  if (m.kind == ABS_LSQ) {
    if (phase != PH_FORWARD) return;
    LsqArgs a;
    a.st = st; a.ri = ri; a.sel = ctx->ctl.sel[par]; a.job = ctx->ctl.job; a.sel_tau = ctx->ctl.sel_tau[par]; a.sel_row0 = ctx->ctl.sel_row0[par]; a.row_idx = ctx->ctl.row_idx[par];
    a.X = ctx->X; a.y = (const float*)ctx->y;
    a.ring = ctx->at<void>(L.ring); a.slot_stride = L.d_pad;
    a.loss = ctx->ctl.loss; a.G = ctx->at<float>(L.G); a.d = m.dims[0];
    if (ctx->lsq_pipe) {
      lsqp::Args q;
      q.st = st; q.ri = ri; q.sel = a.sel; q.job = a.job; q.sel_tau = a.sel_tau;
      q.X = (const __nv_bfloat16*)ctx->X; q.y = a.y; q.ring = (const __nv_bfloat16*)a.ring; q.slot_stride = a.slot_stride;
      q.loss_part = ctx->at<float>(L.row_loss); q.G = a.G; q.d = a.d; q.stages = ctx->lsq_stages;
      q.groups = (m.batch + lsqp::GROUP - 1) / lsqp::GROUP;
      const size_t sm = lsqp::smem_bytes(a.d, ctx->lsq_stages);
      launch_ex(ctx, ABS_KC_LSQ, lsqp::lsq_pipe_kernel, dim3(ctx->lsq_grid), dim3(lsqp::THREADS), sm, q);
    } else if (ctx->lsq_v2) {
      const size_t smw = sizeof(float) * (size_t)a.d;
      const int nv = (a.d + 2047) / 2048;
      if (nv <= 1) launch_ex(ctx, ABS_KC_LSQ, lsq_grad_v2_kernel<T, 1>, dim3(ctx->lsq_grid), dim3(256), smw, a);
      else if (nv == 2) launch_ex(ctx, ABS_KC_LSQ, lsq_grad_v2_kernel<T, 2>, dim3(ctx->lsq_grid), dim3(256), smw, a);
      else launch_ex(ctx, ABS_KC_LSQ, lsq_grad_v2_kernel<T, 4>, dim3(ctx->lsq_grid), dim3(256), smw, a);
    }
    else launch_ex(ctx, ABS_KC_LSQ, lsq_grad_kernel<T>, dim3(ctx->W), dim3(256), 0, a);
    return;
  }
  const int nl = m.n_layers;
  const int row_tiles = L.rows_cap / TM;
  const int row_tiles128 = L.rows_cap / 128;
  const bool gathered = L.path[0] == PATH_TC || L.cnn;     // layer 0 reads act[0]: the gathered rows, or the CNN's features
  const int n_splits = L.P > 0 ? L.P : ctx->W;    // weight-gradient splits (P = 0: one per selected worker)
  LayerArgs la[ABS_MAX_LAYERS];
  for (int l = 0; l < nl; ++l) {
    LayerArgs& a = la[l];
    a.st = st; a.ri = ri; a.tile_slot = ctx->ctl.tile_slot[par]; a.row_idx = ctx->ctl.row_idx[par];
    a.ring = ctx->at<void>(L.gring); a.slot_stride = L.d_pad; a.w_off = L.w_off[l];
    a.in = m.dims[l]; a.out = m.dims[l + 1];
    a.gather = (l == 0 && !gathered);
    a.act_in = (l == 0 && !gathered) ? ctx->X : ctx->at<void>((l == 0 && par) ? L.act0b : L.act[l]);
    a.act_out = (l == nl - 1) ? ctx->at<void>(L.logits) : ctx->at<void>(L.act[l + 1]);
    a.delta_out = ctx->at<void>(L.delta[l + 1]);
    a.delta_in = (l == 0 && !L.cnn) ? nullptr : ctx->at<void>(L.delta[l]);
    a.G = ctx->at<float>(L.G); a.P = L.P;
  }
  // convolution block b of the CNN (0: images -> pooled maps, 1: pooled maps -> features)
  auto conv_args = [&](int b) {
    conv::Args c;
    c.st = st; c.ri = ri; c.tile_slot = ctx->ctl.tile_slot[par]; c.row_idx = ctx->ctl.row_idx[par];
    c.ring = ctx->at<void>(L.gring); c.slot_stride = L.d_pad; c.w_off = L.c_off[b];
    c.Hi = L.cHi[b]; c.Wi = L.cWi[b]; c.Ci = L.cCi[b]; c.k = L.ck; c.Co = L.cCo[b];
    c.in = b == 0 ? ctx->X : ctx->at<void>(L.pool1); c.from_dataset = b == 0 ? 1 : 0;
    c.pooled = b == 0 ? ctx->at<void>(L.pool1) : ctx->at<void>(par ? L.act0b : L.act[0]);
    c.arg = ctx->at<unsigned char>(b == 0 ? L.arg1 : L.arg2);
    c.d_pooled = b == 0 ? ctx->at<void>(L.dpool1) : ctx->at<void>(L.delta[0]);
    c.d_in = b == 0 ? nullptr : ctx->at<void>(L.dpool1);
    c.part = ctx->at<float>(L.cpart[b]);
    c.chunk = L.cchunk;
    return c;
  };
  auto tc_params = [&](int l, int mode) {
    tc::Params p;
    memset(&p, 0, sizeof p);
    p.st = st; p.ri = ri; p.tile_slot = ctx->ctl.tile_slot[par]; p.mode = mode; p.P = L.P;
    p.ring = ctx->at<__nv_bfloat16>(L.gring); p.slot_stride = L.d_pad;
    p.b_off = L.w_off[l] + (size_t)m.dims[l] * m.dims[l + 1];
    return p;
  };
  auto narrow_args = [&](int l) {
    NarrowArgs a;
    a.st = st; a.ri = ri; a.tile_slot = ctx->ctl.tile_slot[par]; a.row_idx = ctx->ctl.row_idx[par]; a.labels = (const int*)ctx->y;
    a.ring = ctx->at<void>(L.gring); a.slot_stride = L.d_pad; a.w_off = L.w_off[l];
    a.in = m.dims[l]; a.C = m.dims[l + 1];
    a.gather = la[l].gather; a.act_in = la[l].act_in;
    a.delta_out = ctx->at<void>(L.delta[l + 1]);
    a.delta_in = (l == 0) ? nullptr : ctx->at<void>(L.delta[l]);
    a.row_loss = L.local_net ? ctx->at<float>(L.row_loss) : ctx->ctl.row_loss; a.G = ctx->at<float>(L.G); a.P = L.P;
    a.rpb = L.narrow_rpb;
    return a;
  };
  if (phase == PH_GATHER && L.cnn) {
    // Eq. 2 forward through the two convolution blocks: the features are the input rows of layer 0
    for (int b = 0; b < 2; ++b) {
      const conv::Args c = conv_args(b);
      launch_ex(ctx, ABS_KC_CONV, conv::conv_block_fwd_kernel<T>, dim3(L.rows_cap), dim3(conv::THREADS),
                conv::fwd_smem_bytes(c.Hi, c.Wi, c.Ci, c.k, c.Co), c);
    }
    return;
  }
  if (phase == PH_GATHER) {
    if (gathered)
      launch_on(ctx, ctx->overlap ? ctx->side : s, ABS_KC_GATHER, gather_rows_kernel, dim3(ctx->sm_count * 8), dim3(256), 0,
                st, ri, ctx->ctl.row_idx[par], (const __nv_bfloat16*)ctx->X, ctx->at<__nv_bfloat16>(par ? L.act0b : L.act[0]), m.dims[0]);
    return;
  }
  // ---- forward (Eq. 2 at the model version each worker holds)
  for (int l = 0; l < nl && phase == PH_FORWARD; ++l) {
    const bool last = l == nl - 1;
    if (L.path[l] == PATH_TC) {
      tc::Params p = tc_params(l, tc::FWD);
      p.N_total = la[l].out; p.K_total = la[l].in;
      p.out_bf16 = (__nv_bfloat16*)la[l].act_out;
      p.relu_bits = L.bits[l + 1] ? ctx->at<uint32_t>(L.bits[l + 1]) : nullptr;
      p.mask_words = (la[l].out + 31) / 32;
      const int bn = L.bn_fwd[l];
      const CUtensorMap& amap = (l == 0 && par) ? ctx->tcl[l].fwd_a_odd : ctx->tcl[l].fwd_a;
      const int tiles = (row_tiles128 / L.cg_fwd[l]) * ((la[l].out + bn - 1) / bn);
      launch_tc_bn(ctx, bn, L.cg_fwd[l], ABS_KC_FWD, amap, ctx->tcl[l].fwd_b, ctx->tcl[l].fwd_out, p, tiles);
    } else if (L.path[l] == PATH_NARROW) {
      NarrowArgs a = narrow_args(l);
      if (L.fused_R) {
        int R = L.fused_R;
        const size_t sm = sizeof(T) * ((size_t)R * a.in + (size_t)a.C * (a.in + 8) + (size_t)(a.in + 1) * a.C) + 64 +
                          sizeof(float) * (size_t)R * NARROW_MAX_C;
        float* part = ctx->at<float>(L.red);
        float* dstw = ctx->at<float>(L.G) + L.w_off[l];
        const int len = (a.in + 1) * a.C, has_dgrad = l > 0 ? 1 : 0;
        if (L.out_mma) {
          const dim3 og(L.rows_cap / outl::ROWS), ob(outl::THREADS);
          const size_t osm = outl::smem_bytes(a.in, a.C);
          if (a.in == 128) launch_ex(ctx, ABS_KC_OUTPUT, outl::out_layer_mma_kernel<1>, og, ob, osm, a, part, has_dgrad);
          else if (a.in == 256) launch_ex(ctx, ABS_KC_OUTPUT, outl::out_layer_mma_kernel<2>, og, ob, osm, a, part, has_dgrad);
          else if (a.in == 512) launch_ex(ctx, ABS_KC_OUTPUT, outl::out_layer_mma_kernel<4>, og, ob, osm, a, part, has_dgrad);
          else launch_ex(ctx, ABS_KC_OUTPUT, outl::out_layer_mma_kernel<8>, og, ob, osm, a, part, has_dgrad);
          R = outl::ROWS;
        } else if (a.C == 10) {
          const size_t smc = sizeof(T) * ((size_t)R * a.in + (size_t)(a.in + 1) * 10) + 32 +
                             sizeof(float) * ((size_t)10 * (a.in + 4) + (size_t)R * 10);
          launch_ex(ctx, ABS_KC_OUTPUT, narrow_fused_cc_kernel<T, 10>, dim3(L.rows_cap / R), dim3(256), smc, a, part, R, has_dgrad);
        } else {
          launch_ex(ctx, ABS_KC_OUTPUT, narrow_fused_kernel<T>, dim3(L.rows_cap / R), dim3(256), sm, a, part, R, has_dgrad);
        }
        // U = 1: the chunk partials are added up by extra blocks of the Eq. 3 kernel (one launch less)
        if (L.local_net)
          launch_ex(ctx, ABS_KC_OUTPUT, lnet::chunk_reduce_worker_kernel, dim3((len + 255) / 256, ctx->W), dim3(256), 0, st, ri, part, len,
                    dstw, L.d_pad, R, L.RBp);
      } else if (a.in % 8 == 0) {
        const size_t sm = sizeof(T) * (size_t)a.in * a.C + sizeof(float) * a.C;
        launch_ex(ctx, ABS_KC_OUTPUT, narrow_fwd_loss_v8_kernel<T>, dim3(L.rows_cap / NARROW_ROWS), dim3(256), sm, a);
      } else {
        const size_t sm = sizeof(float) * ((size_t)a.in * a.C + a.C);
        launch_ex(ctx, ABS_KC_OUTPUT, narrow_fwd_loss_kernel<T>, dim3(L.rows_cap / L.narrow_rpb), dim3(256), sm, a);
      }
    } else {
      dim3 grid((la[l].out + TN - 1) / TN, row_tiles);
      const int cls = last ? ABS_KC_OUTPUT : ABS_KC_FWD;
      if (last) launch_ex(ctx, cls, simt_fwd_kernel<T, true>, dim3(grid), dim3(256), 0, la[l]);
      else launch_ex(ctx, cls, simt_fwd_kernel<T, false>, dim3(grid), dim3(256), 0, la[l]);
      if (last) {
        LossArgs lo;
        lo.st = st; lo.ri = ri; lo.tile_slot = ctx->ctl.tile_slot[par]; lo.row_idx = ctx->ctl.row_idx[par]; lo.labels = (const int*)ctx->y;
        lo.logits = ctx->at<float>(L.logits); lo.delta = ctx->at<void>(L.delta[nl]);
        lo.row_loss = L.local_net ? ctx->at<float>(L.row_loss) : ctx->ctl.row_loss; lo.C = m.dims[nl];
        launch_ex(ctx, ABS_KC_OUTPUT, net_loss_kernel<T>, dim3((L.rows_cap + 255) / 256), dim3(256), 0, lo);
      }
    }
  }
  // ---- backward: deltas, then the weight gradients summed over all selected workers (Eq. 3)
  for (int l = nl - 1; l >= 0 && phase == PH_BACKWARD; --l) {
    if (L.path[l] == PATH_TC) {
      tc::Params pd = tc_params(l, tc::DGRAD);
      pd.N_total = la[l].in; pd.K_total = la[l].out;
      pd.mask_src = (const __nv_bfloat16*)la[l].act_in;
      pd.mask_bits = L.bits[l] ? ctx->at<uint32_t>(L.bits[l]) : nullptr;
      pd.mask_words = (la[l].in + 31) / 32;
      pd.out_bf16 = (__nv_bfloat16*)la[l].delta_in;
      if (l > 0 && L.bias_colsum[l - 1]) pd.colsum = ctx->at<float>(L.colsum[l - 1]);   // bias gradient of the layer below
      const int bnd = L.bn_dg[l];
      const int dg_tiles = (row_tiles128 / std::max(1, L.cg_dg[l])) * ((la[l].in + std::max(1, bnd) - 1) / std::max(1, bnd));
      tc::Params p = tc_params(l, tc::WGRAD);
      p.M_total = la[l].in + 1; p.N_total = la[l].out;     // row `in` of the result is the bias gradient
      p.out_f32 = ctx->at<float>(L.G) + L.w_off[l];
      p.no_bias_tile = L.bias_colsum[l] ? 1 : 0;
      const int bias_tiles = L.bias_colsum[l] ? 0 : 1;
      if (l > 0 && L.pair_bwd[l]) {
        // the layer's delta back-propagation shares the weight gradient's launch (same tile width)
        const TcProblem second = {&ctx->tcl[l].dg_a, &ctx->tcl[l].dg_b, &ctx->tcl[l].dg_out, &pd, dg_tiles};
        launch_tc_bn(ctx, bnd, 1, ABS_KC_WGRAD, ctx->tcl[l].wg_a, ctx->tcl[l].wg_b, ctx->tcl[l].wg_out, p,
                     ((la[l].in + 127) / 128 + bias_tiles) * ((la[l].out + bnd - 1) / bnd) * n_splits, &second);
        continue;
      }
      if (l > 0 || L.cnn)
        launch_tc_bn(ctx, bnd, L.cg_dg[l], ABS_KC_DGRAD, ctx->tcl[l].dg_a, ctx->tcl[l].dg_b, ctx->tcl[l].dg_out, pd, dg_tiles);
      const int bn = L.bn_wg[l];
      const int tmw = 128 * L.cg_wg[l];
      launch_tc_bn(ctx, bn, L.cg_wg[l], ABS_KC_WGRAD, (l == 0 && par) ? ctx->tcl[l].wg_a_odd : ctx->tcl[l].wg_a, ctx->tcl[l].wg_b, ctx->tcl[l].wg_out, p,
                   ((la[l].in + tmw - 1) / tmw + bias_tiles) * ((la[l].out + bn - 1) / bn) * n_splits);
    } else if (L.path[l] == PATH_NARROW && L.fused_R) {
      // forward, loss, delta of the layer below and the gradient were all done by the fused kernel
    } else if (L.path[l] == PATH_NARROW) {
      NarrowArgs a = narrow_args(l);
      if (l > 0) {
        if (a.in % 8 == 0) {
          const size_t sm = sizeof(T) * (size_t)a.in * a.C + sizeof(float) * NARROW_ROWS * a.C;
          launch_ex(ctx, ABS_KC_OUTPUT, narrow_dgrad_v8_kernel<T>, dim3(L.rows_cap / NARROW_ROWS), dim3(256), sm, a);
        } else {
          const size_t sm = sizeof(float) * ((size_t)a.in * a.C + 64 * a.C);
          launch_ex(ctx, ABS_KC_OUTPUT, narrow_dgrad_kernel<T>, dim3(L.rows_cap / L.narrow_rpb), dim3(256), sm, a);
        }
      }
      // weight gradient: per-chunk partial sums, then one ordered sum over the chunks into partial 0
      float* part = ctx->at<float>(L.red);
      float* dstw = ctx->at<float>(L.G) + L.w_off[l];
      const int len = (a.in + 1) * a.C;
      launch_ex(ctx, ABS_KC_OUTPUT, narrow_wgrad_chunk_kernel<T>, dim3(L.rows_cap / L.narrow_rpb), dim3(256), 0, a, part);
      if (L.local_net)
        launch_ex(ctx, ABS_KC_OUTPUT, lnet::chunk_reduce_worker_kernel, dim3((len + 255) / 256, ctx->W), dim3(256), 0, st, ri, part, len,
                  dstw, L.d_pad, 64, L.RBp);
      else
        launch_ex(ctx, ABS_KC_OUTPUT, chunk_reduce_kernel, dim3((len + 31) / 32), dim3(256), 0, st, ri, part, len, dstw, L.narrow_rpb);
    } else {
      const bool last = l == nl - 1;
      if (l > 0 || L.cnn) {
        dim3 grid((la[l].in + TN - 1) / TN, row_tiles);
        launch_ex(ctx, last ? ABS_KC_OUTPUT : ABS_KC_DGRAD, simt_dgrad_kernel<T>, dim3(grid), dim3(256), 0, la[l]);
      }
      dim3 gridw((la[l].out + TN - 1) / TN, (la[l].in + 1 + TM - 1) / TM, n_splits);
      launch_ex(ctx, last ? ABS_KC_OUTPUT : ABS_KC_WGRAD, simt_wgrad_kernel<T>, dim3(gridw), dim3(256), 0, la[l]);
    }
  }
  // ---- CNN: back through the convolution blocks (second, then first); their weight gradients are
  // per-chunk sums that a fixed-order reduction adds up into partial 0 of the gradient vector
  for (int b = 1; b >= 0 && phase == PH_BACKWARD && L.cnn; --b) {
    const conv::Args c = conv_args(b);
    if (b == 1)      // delta of the first block's pooled maps (one CTA per row)
      launch_ex(ctx, ABS_KC_CONV, conv::conv_block_dgrad_kernel<T>, dim3(L.rows_cap), dim3(conv::THREADS),
                conv::dgrad_smem_bytes(c.Hi, c.Wi, c.Ci, c.k, c.Co), c);
    launch_ex(ctx, ABS_KC_CONV, conv::conv_block_wgrad_kernel<T>, dim3(L.rows_cap / L.cchunk), dim3(conv::THREADS),
              conv::wgrad_smem_bytes(c.Hi, c.Wi, c.Ci, c.k, c.Co), c);
    launch_ex(ctx, ABS_KC_CONV, chunk_reduce_kernel, dim3(((int)L.c_len[b] + 31) / 32), dim3(256), 0, st, ri, c.part, (int)L.c_len[b],
              ctx->at<float>(L.G) + L.c_off[b], L.cchunk);
  }
}

template <typename T>
void enqueue_update(abs_ctx* ctx, int par) {
  const Layout& L = ctx->L;
  RoundInfo* ri = ctx->at<RoundInfo>(L.ri) + par;
  if (ctx->lsq_v2) {
    LsqUpdateArgs q;
    q.st = ctx->at<DevState>(L.st); q.ri = ri; q.job = ctx->ctl.job; q.next_dur = nullptr; q.dur_job = ctx->ctl.dur_job;   // durations: control kernel
    q.master = ctx->at<float>(L.master); q.ring = ctx->at<void>(L.ring); q.G = ctx->at<float>(L.G);
    q.d_pad = L.d_pad; q.d = ctx->m.dims[0]; q.P = ctx->lsq_grid; q.lr = ctx->m.lr;
    q.loss_part = ctx->lsq_pipe ? ctx->at<float>(L.row_loss) : nullptr;
    q.loss = ctx->ctl.loss; q.groups = (ctx->m.batch + lsqp::GROUP - 1) / lsqp::GROUP;
    const int blocks = std::max((q.d + 31) / 32, (ctx->W + 31) / 32);
    launch_ex(ctx, ABS_KC_UPDATE, lsq_update_kernel<T>, dim3(blocks), dim3(256), 0, q);
    return;
  }
  UpdateArgs u;
  u.st = ctx->at<DevState>(L.st); u.ri = ri; u.master = ctx->at<float>(L.master); u.ring = ctx->at<void>(L.ring);
  u.G = ctx->at<float>(L.G); u.d_pad = L.d_pad; u.P = L.P; u.lr = ctx->m.lr;
  u.sel_tau = ctx->ctl.sel_tau[par];
  // for the latency-bound models (always one stream) the Eq. 3 kernel also prepares the next job
  // durations (its first warps); tensor-core networks keep a small kernel of their own for that
  // job durations are prepared by the control kernel, except on the local-step paths
  const bool look = ctx->local_sgd || (L.local_net && !L.any_tc);
  u.job = ctx->ctl.job; u.next_dur = ctx->ctl.next_dur; u.dur_job = ctx->ctl.dur_job;
  // one wave of resident blocks striding over the vector (a partly filled second wave would only add a tail)
  const size_t n4 = L.d_pad / 4;
  int blocks = (int)std::max<size_t>(std::min<size_t>((n4 + 255) / 256, (size_t)ctx->sm_count * ctx->upd_blocks_per_sm), (size_t)(ctx->W + 31) / 32);
  u.n_regions = 0; u.n_main_blocks = blocks;
  memset(u.region, 0, sizeof u.region);
  auto add_region = [&](const float* part, int len, int chunk_rows, size_t off) {
    UpdateArgs::Region& R = u.region[u.n_regions++];
    R.part = part; R.len = len; R.chunk_rows = chunk_rows; R.off = off; R.first_block = blocks - u.n_main_blocks;
    blocks += (len + 31) / 32;
  };
  const int last = ctx->m.n_layers - 1;
  if (ctx->m.kind != ABS_LSQ && L.fused_R && L.path[last] == PATH_NARROW && !L.local_net && !ctx->local_sgd)
    // the fused output-layer kernel left its gradient as per-chunk partial sums
    add_region(ctx->at<float>(L.red), (ctx->m.dims[last] + 1) * ctx->m.dims[last + 1], L.out_mma ? outl::ROWS : L.fused_R, L.w_off[last]);
  for (int l = 0; l < ctx->m.n_layers && u.n_regions < UpdateArgs::MAX_REGIONS; ++l)
    if (L.bias_colsum[l])     // bias gradient as column sums per 32 rows, left by the back-propagation of the layer above
      add_region(ctx->at<float>(L.colsum[l]), ctx->m.dims[l + 1], 32, L.w_off[l] + (size_t)ctx->m.dims[l] * ctx->m.dims[l + 1]);
  if (look) launch_ex(ctx, ABS_KC_UPDATE, update_kernel<T, true>, dim3(blocks), dim3(256), 0, u);
  else launch_ex(ctx, ABS_KC_UPDATE, update_kernel<T, false>, dim3(blocks), dim3(256), 0, u);
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
    case ST_STALE:
      ctx->sticky = ABS_ESTALE;
      return fail(ABS_ESTALE, "round %d: an upload older than the staleness bound arrived (no forced restarts); "
                  "%d completed rounds stay valid", h.t, h.t);
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
  make_layout(model, W, staleness_bound + (model->restart_rule == ABS_RESTART_EQ6 ? 1 : 0), &L);
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
  if (model->local_steps < 1 || model->local_steps > 1024)
    return fail(ABS_EINVAL, "local_steps %d outside [1, 1024]", model->local_steps);
  if (model->local_steps > 1) {
    // U > 1: the worker's local model lives in shared memory; single-layer models only
    const bool single = model->kind != ABS_MLP || model->n_layers == 1;
    const int C = model->kind == ABS_LSQ ? 1 : model->dims[1];
    const size_t n_par = model->kind == ABS_LSQ ? (size_t)model->dims[0] : (size_t)model->dims[0] * C + C;
    if (single && (C > local::MAX_C || n_par > (size_t)local::MAX_PARAMS || (size_t)model->batch * C > (size_t)local::MAX_BC))
      return fail(ABS_EUNSUPPORTED, "local_steps > 1 needs at most %d classes, %d parameters and batch x classes <= %d",
                  local::MAX_C, local::MAX_PARAMS, local::MAX_BC);
  }
  if (K0 < 1 || K0 > W) return fail(ABS_EINVAL, "K0 %d outside [1, W]", K0);
  if (model->k_mode != ABS_K_ADAPTIVE && model->k_mode != ABS_K_FIXED) return fail(ABS_EINVAL, "k_mode");
  if (model->bound_mode != ABS_BOUND_ADAPTIVE && model->bound_mode != ABS_BOUND_FIXED &&
      model->bound_mode != ABS_BOUND_OFFSET)
    return fail(ABS_EINVAL, "bound_mode");
  if (model->bound_mode == ABS_BOUND_OFFSET) {
    if (model->bound_offset < -ABS_MAX_WORKERS || model->bound_offset > ABS_MAX_BOUND)
      return fail(ABS_EINVAL, "bound_offset %d out of range", model->bound_offset);
    if (std::max(1, W / K0 + model->bound_offset) > staleness_bound)
      return fail(ABS_EINVAL, "staleness_bound %d is below the initial threshold floor(N/K0) + a = %d",
                  staleness_bound, W / K0 + model->bound_offset);
  }
  if (!(model->lr >= 0.f) || !std::isfinite(model->lr)) return fail(ABS_EINVAL, "lr");
  if (!td) return fail(ABS_EINVAL, "time_dist is null");
  if (td->kind < ABS_T_CONST || td->kind > ABS_T_GAMMA) return fail(ABS_EUNSUPPORTED, "time_dist kind %d", td->kind);
  if ((td->kind == ABS_T_EXP || td->kind == ABS_T_SHIFTED_EXP || td->kind == ABS_T_GAMMA) && !(td->rate > 0.0)) return fail(ABS_EINVAL, "rate must be > 0");
  if ((td->kind == ABS_T_CONST || td->kind == ABS_T_SHIFTED_EXP || td->kind == ABS_T_GAMMA) && !(td->shift >= 0.0)) return fail(ABS_EINVAL, "shift must be >= 0");
  if (td->kind == ABS_T_GAMMA && (td->shape < 1 || td->shape > 64)) return fail(ABS_EINVAL, "gamma shape %d outside [1, 64]", td->shape);
  if (td->kind == ABS_T_PARETO2 && !(td->scale > 0.0)) return fail(ABS_EINVAL, "scale must be > 0");
  if (td->slow_mod < 0 || (td->slow_mod > 0 && (td->slow_rem < 0 || td->slow_rem >= td->slow_mod)))
    return fail(ABS_EINVAL, "slow class");
  if (td->slow_mod > 0 && !(td->slow_factor > 0.0)) return fail(ABS_EINVAL, "slow_factor must be > 0");
  if (!model->X || !model->y || !model->w0) return fail(ABS_EINVAL, "X, y and w0 must be non-null");
  if (!model->workspace) return fail(ABS_EINVAL, "workspace is null");
  if (((uintptr_t)model->workspace & 255) != 0) return fail(ABS_EINVAL, "workspace must be 256-byte aligned");
  if (!model->data_on_host && (((uintptr_t)model->X & 15) != 0 || ((uintptr_t)model->y & 3) != 0))
    return fail(ABS_EINVAL, "X must be 16-byte aligned, y 4-byte aligned");
  // Eq. 6 as printed lets a consumed gradient be one round older: one more ring slot, same threshold
  const int literal = model->restart_rule == ABS_RESTART_EQ6 ? 1 : 0;
  const int S_ring = staleness_bound + literal;
  Layout L;
  make_layout(model, W, S_ring, &L);
  if (model->workspace_bytes < L.total)
    return fail(ABS_ENOSPACE, "workspace has %zu bytes, %zu needed", model->workspace_bytes, L.total);

  ctx = new (std::nothrow) abs_ctx();
  if (!ctx) return fail(ABS_EINVAL, "out of host memory");
  ctx->m = *model; ctx->L = L; ctx->W = W; ctx->K0 = K0; ctx->S = S_ring;
  ctx->stream = (cudaStream_t)model->stream;
  ctx->ws = (char*)model->workspace;
  cudaStream_t s = ctx->stream;
  auto bail = [&](int code) { delete ctx; return code; };

  // everything except the dataset copy starts from zero (gradient padding must stay zero)
  const size_t zero_bytes = model->data_on_host ? L.data_X : L.total;
  cudaError_t e = cudaMemsetAsync(ctx->ws, 0, zero_bytes, s);
  if (e != cudaSuccess) return bail(cuda_fail(nullptr, e, "cudaMemsetAsync(workspace)"));
  if (model->data_on_host) {
    e = cudaMemcpyAsync(ctx->ws + L.data_X, model->X, L.esz * (size_t)model->n_samples * L.x_len, cudaMemcpyHostToDevice, s);
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
  for (int b = 0; b < 2 && L.cnn; ++b) {
    e = cudaMemcpyAsync(ctx->at<float>(L.master) + L.c_off[b], model->w0 + L.c_src[b], 4 * L.c_len[b], cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return bail(cuda_fail(nullptr, e, "w0 copy"));
  }
  DevState h;
  memset(&h, 0, sizeof h);
  h.W = W; h.K0 = K0; h.S = S_ring; h.B = model->batch; h.RB = L.RB;
  h.theta_cap = staleness_bound; h.literal_eq6 = literal;
  h.no_restart = model->restart_rule == ABS_RESTART_NONE ? 1 : 0;
  // staleness-aware step size: applied to the delta rows / residuals by the gradient kernels, except
  // with local steps on a network, whose local copies need the plain gradient sums (there Eq. 3
  // weights the uploads)
  h.sa_penalty = model->sa_penalty ? (L.local_net ? 2 : 1) : 0;
  h.k_mode = model->k_mode; h.bound_mode = model->bound_mode; h.max_rounds = model->max_rounds;
  h.n_samples = model->n_samples;
  h.key0 = (uint32_t)(seed & 0xffffffffull); h.key1 = (uint32_t)(seed >> 32);
  h.dist.kind = td->kind; h.dist.shift = td->shift; h.dist.rate = td->rate; h.dist.scale = td->scale;
  h.dist.slow_mod = td->slow_mod; h.dist.slow_rem = td->slow_rem; h.dist.slow_factor = td->slow_factor;
  h.dist.shape = td->kind == ABS_T_GAMMA ? td->shape : 1;
  h.bound_offset = model->bound_offset;
  h.K = K0; h.theta = staleness_bound; h.comm = (u64)W;
  e = cudaMemcpyAsync(ctx->at<DevState>(L.st), &h, sizeof h, cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return bail(cuda_fail(nullptr, e, "state copy"));

  CtlArgs& c = ctx->ctl;
  c.st = ctx->at<DevState>(L.st);
  c.c = ctx->at<u64>(L.c); c.version = ctx->at<int>(L.version); c.job = ctx->at<int>(L.job);
  c.next_dur = ctx->at<u64>(L.next_dur); c.dur_job = ctx->at<int>(L.dur_job);
  c.ri = ctx->at<RoundInfo>(L.ri);
  for (int q = 0; q < 2; ++q) {
    c.sel[q] = ctx->at<int>(L.sel[q]); c.sel_tau[q] = ctx->at<int>(L.sel_tau[q]); c.sel_row0[q] = ctx->at<int>(L.sel_row0[q]);
    c.row_idx[q] = ctx->at<int>(L.row_idx[q]); c.tile_slot[q] = ctx->at<int>(L.tile_slot[q]);
  }
  c.loss = ctx->at<float>(L.loss);
  c.loss_part = nullptr; c.loss_groups = 0;
  // with local steps a worker's loss is uploaded whole (no per-row losses, no row layout)
  c.row_loss = (model->kind == ABS_LSQ || model->local_steps > 1) ? nullptr : ctx->at<float>(L.row_loss);
  c.tr_K = ctx->at<int>(L.tr_K); c.tr_R = ctx->at<int>(L.tr_R); c.tr_theta = ctx->at<int>(L.tr_theta);
  c.tr_T = ctx->at<u64>(L.tr_T); c.tr_loss = ctx->at<float>(L.tr_loss); c.tr_comm = ctx->at<u64>(L.tr_comm);
  c.tr_sel_off = ctx->at<i64>(L.tr_sel_off); c.tr_rst_off = ctx->at<i64>(L.tr_rst_off);
  c.tr_sel_id = ctx->at<int>(L.tr_sel_id); c.tr_sel_tau = ctx->at<int>(L.tr_sel_tau);
  c.tr_sel_loss = ctx->at<float>(L.tr_sel_loss); c.tr_rst_id = ctx->at<int>(L.tr_rst_id);

  {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
      ctx->sm_count = sms;
  }
  {
    const cudaError_t ea = cudaFuncSetAttribute(abs_ctl_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)sizeof(CtlShared));
    if (ea != cudaSuccess) return bail(cuda_fail(nullptr, ea, "cudaFuncSetAttribute(abs_ctl_kernel)"));
    const cudaError_t eb = cudaFuncSetAttribute(abs_ctl_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)sizeof(CtlShared));
    if (eb != cudaSuccess) return bail(cuda_fail(nullptr, eb, "cudaFuncSetAttribute(abs_ctl_small_kernel)"));
  }
  if (L.out_mma) {
    const int osm = (int)outl::smem_bytes(model->dims[model->n_layers - 1], model->dims[model->n_layers]);
    cudaError_t eo = cudaFuncSetAttribute(outl::out_layer_mma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, osm);
    if (eo == cudaSuccess) eo = cudaFuncSetAttribute(outl::out_layer_mma_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, osm);
    if (eo == cudaSuccess) eo = cudaFuncSetAttribute(outl::out_layer_mma_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, osm);
    if (eo == cudaSuccess) eo = cudaFuncSetAttribute(outl::out_layer_mma_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, osm);
    if (eo != cudaSuccess) return bail(cuda_fail(nullptr, eo, "cudaFuncSetAttribute(out_layer_mma_kernel)"));
  }
  if (L.fused_R) {
    cudaError_t ef = cudaFuncSetAttribute(narrow_fused_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
    if (ef == cudaSuccess)
      ef = cudaFuncSetAttribute(narrow_fused_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
    if (ef == cudaSuccess)
      ef = cudaFuncSetAttribute(narrow_fused_cc_kernel<float, 10>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
    if (ef == cudaSuccess)
      ef = cudaFuncSetAttribute(narrow_fused_cc_kernel<__nv_bfloat16, 10>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
    if (ef != cudaSuccess) return bail(cuda_fail(nullptr, ef, "cudaFuncSetAttribute(narrow_fused_kernel)"));
  }
  if (model->local_steps > 1 && !L.local_net) {
    const int C = model->kind == ABS_LSQ ? 1 : model->dims[1];
    const int n_par = model->kind == ABS_LSQ ? model->dims[0] : model->dims[0] * C + C;
    const int sm = (int)local::smem_bytes(n_par, model->batch, C);
    cudaError_t el = cudaFuncSetAttribute(local::local_sgd_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
    if (el == cudaSuccess) el = cudaFuncSetAttribute(local::local_sgd_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
    if (el != cudaSuccess) return bail(cuda_fail(nullptr, el, "cudaFuncSetAttribute(local_sgd_kernel)"));
    ctx->local_sgd = true;
  }
  if (!ctx->local_sgd && model->kind == ABS_LSQ && model->dims[0] % 8 == 0 && model->dims[0] <= LSQ_MAX_D) {
    ctx->lsq_v2 = true;
    ctx->lsq_grid = std::min(W, 2 * ctx->sm_count);
    // bf16 rows of up to 8 KB: stream them through shared memory with bulk copies, one CTA per SM
    if (model->dtype == ABS_BF16_FP32MASTER && model->dims[0] <= 4096 && !(model->flags & ABS_FLAG_NO_BULK_PIPELINE)) {
      int stages = lsqp::MAX_STAGES;
      while (stages >= 2 && lsqp::smem_bytes(model->dims[0], stages) > 227 * 1024) --stages;
      if (stages >= 2) {
        const int sm = (int)lsqp::smem_bytes(model->dims[0], stages);
        cudaError_t ep = cudaFuncSetAttribute(lsqp::lsq_pipe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
        if (ep != cudaSuccess) return bail(cuda_fail(nullptr, ep, "cudaFuncSetAttribute(lsq_pipe_kernel)"));
        ctx->lsq_pipe = true;
        ctx->lsq_stages = stages;
        ctx->lsq_grid = std::min(W, ctx->sm_count);
      }
    }
  }
  if (!ctx->local_sgd && model->kind == ABS_LSQ && !(model->flags & ABS_FLAG_NO_PERSISTENT) && model->dims[0] % 8 == 0 &&
      model->dims[0] <= LSQ_ROUNDS_MAX_D && W <= LSQ_ROUNDS_NTG && (size_t)W * model->batch <= LSQ_ROUNDS_MAX_ROWS &&
      (size_t)(S_ring + 1) * model->dims[0] * 4 <= 64 * 1024) {
    const size_t sm = lsq_rounds_smem(S_ring, model->dims[0]);
    cudaError_t er = cudaFuncSetAttribute(abs_lsq_rounds_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (er == cudaSuccess)
      er = cudaFuncSetAttribute(abs_lsq_rounds_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (er != cudaSuccess) return bail(cuda_fail(nullptr, er, "cudaFuncSetAttribute(abs_lsq_rounds_kernel)"));
    ctx->lsq_rounds = true;
  }
  if (ctx->lsq_pipe && !ctx->lsq_rounds) {
    // the pipeline kernel leaves per-group loss sums: the control step finishes the uploaded losses
    // itself (it runs next to the Eq. 3 kernel, which finishes them too, for its own divergence check)
    ctx->ctl.loss_part = ctx->at<float>(L.row_loss);
    ctx->ctl.loss_groups = (model->batch + lsqp::GROUP - 1) / lsqp::GROUP;
  }
  rc = setup_tc(ctx);
  if (rc != ABS_OK) return bail(rc);
  {
    int occ = 0;
    cudaError_t eo;
    if (model->dtype == ABS_FP32)
      eo = L.any_tc ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, update_kernel<float, false>, 256, 0)
                    : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, update_kernel<float, true>, 256, 0);
    else
      eo = L.any_tc ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, update_kernel<__nv_bfloat16, false>, 256, 0)
                    : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, update_kernel<__nv_bfloat16, true>, 256, 0);
    if (eo != cudaSuccess) return bail(cuda_fail(nullptr, eo, "cudaOccupancyMaxActiveBlocksPerMultiprocessor(update_kernel)"));
    ctx->upd_blocks_per_sm = std::max(1, std::min(occ, 8));
  }
  // worth it only when a round has a long backward pass to hide behind (tensor-core networks);
  // for the latency-bound models the cross-stream events cost more than they hide
  if (L.cnn) {
    size_t need = 0;
    for (int b = 0; b < 2; ++b)
      need = std::max(need, std::max(conv::fwd_smem_bytes(L.cHi[b], L.cWi[b], L.cCi[b], L.ck, L.cCo[b]),
                                     conv::bwd_smem_bytes(L.cHi[b], L.cWi[b], L.cCi[b], L.ck, L.cCo[b])));
    cudaError_t ec = cudaFuncSetAttribute(conv::conv_block_fwd_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
    if (ec == cudaSuccess) ec = cudaFuncSetAttribute(conv::conv_block_fwd_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
    if (ec == cudaSuccess) ec = cudaFuncSetAttribute(conv::conv_block_wgrad_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
    if (ec == cudaSuccess) ec = cudaFuncSetAttribute(conv::conv_block_wgrad_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
    if (ec == cudaSuccess) ec = cudaFuncSetAttribute(conv::conv_block_dgrad_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
    if (ec == cudaSuccess) ec = cudaFuncSetAttribute(conv::conv_block_dgrad_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
    if (ec != cudaSuccess) return bail(cuda_fail(nullptr, ec, "cudaFuncSetAttribute(conv_block kernels)"));
  }
  if (!(model->flags & ABS_FLAG_NO_OVERLAP) && L.any_tc && !L.local_net && !L.cnn) {
    cudaError_t es = cudaStreamCreateWithFlags(&ctx->side, cudaStreamNonBlocking);
    if (es == cudaSuccess) es = cudaEventCreateWithFlags(&ctx->ev_loss, cudaEventDisableTiming);
    if (es == cudaSuccess) es = cudaEventCreateWithFlags(&ctx->ev_ctl, cudaEventDisableTiming);
    if (es != cudaSuccess) return bail(cuda_fail(nullptr, es, "side stream / events"));
    ctx->overlap = true;
  }
  abs_init_state_kernel<<<(W + 31) / 32, 32, 0, s>>>(c);
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
  const size_t csm = sizeof(CtlShared);
  void (*ctl_kernel)(CtlArgs, int, int, int, int, int) = ctx->W <= 256 ? abs_ctl_small_kernel : abs_ctl_kernel;
  const int ctl_threads = ctx->W <= 256 ? 256 : 1024;
  const int times_blocks = (ctx->W + 31) / 32;
  const DevState* stc = ctx->at<DevState>(ctx->L.st);
  auto gradient = [&](int par, int phase) {
    if (f32) enqueue_gradient<float>(ctx, par, phase);
    else enqueue_gradient<__nv_bfloat16>(ctx, par, phase);
  };
  auto update = [&](int par) {
    if (f32) enqueue_update<float>(ctx, par);
    else enqueue_update<__nv_bfloat16>(ctx, par);
  };
  if (n > 0 && ctx->local_sgd) {
    local::Args q;
    q.st = ctx->at<DevState>(ctx->L.st);
    q.sel = nullptr; q.sel_tau = nullptr; q.ri = nullptr;
    q.job = ctx->ctl.job; q.X = ctx->X; q.y = ctx->y;
    q.ring = ctx->at<void>(ctx->L.ring); q.slot_stride = ctx->L.d_pad;
    q.loss = ctx->ctl.loss; q.G = ctx->at<float>(ctx->L.G);
    q.lsq = ctx->m.kind == ABS_LSQ ? 1 : 0;
    q.in = ctx->m.dims[0]; q.C = q.lsq ? 1 : ctx->m.dims[1]; q.U = ctx->m.local_steps; q.lr = ctx->m.lr;
    const size_t sm = local::smem_bytes(q.lsq ? q.in : q.in * q.C + q.C, ctx->m.batch, q.C);
    const int nt = local::threads_for(q.lsq ? q.in : q.in * q.C + q.C);
    for (int r = 0; r < n; ++r) {
      const int t = ctx->rounds_enqueued + r, par = t & 1;
      launch_ex(ctx, ABS_KC_CTL, ctl_kernel, dim3(1), dim3(ctl_threads), csm, ctx->ctl, 1, 1, t, 0, 0);
      q.ri = ctx->at<RoundInfo>(ctx->L.ri) + par;
      q.sel = ctx->ctl.sel[par]; q.sel_tau = ctx->ctl.sel_tau[par];
      if (f32) launch_ex(ctx, ABS_KC_LSQ, local::local_sgd_kernel<float>, dim3(ctx->W), dim3(nt), sm, q);
      else launch_ex(ctx, ABS_KC_LSQ, local::local_sgd_kernel<__nv_bfloat16>, dim3(ctx->W), dim3(nt), sm, q);
      update(par);
    }
    launch_ex(ctx, ABS_KC_CTL, ctl_kernel, dim3(1), dim3(ctl_threads), csm, ctx->ctl, 1, 0, ctx->rounds_enqueued + n, 0, 0);
  } else if (n > 0 && ctx->L.local_net) {
    // U > 1 on a multi-layer network: per round, the workers' copies are set up, then every local
    // step is one pass of the gradient kernels over the private copies (which add each worker's
    // gradient to its upload) followed by the refresh of the copies
    const Layout& L = ctx->L;
    lnet::Args q;
    q.st = ctx->at<DevState>(L.st);
    q.job = ctx->ctl.job;
    q.ring = ctx->at<void>(L.ring);
    q.priv = ctx->at<void>(L.priv); q.gsum = ctx->at<float>(L.G);
    q.row_loss = ctx->at<float>(L.row_loss);
    q.loss_acc = ctx->at<float>(L.loss_acc); q.loss = ctx->ctl.loss;
    q.d_pad = L.d_pad; q.RBp = L.RBp; q.U = ctx->m.local_steps; q.lr = ctx->m.lr;
    const int bx = (int)std::max<size_t>(1, std::min<size_t>((L.d_pad / 4 + 1023) / 1024, 64));
    for (int r = 0; r < n; ++r) {
      const int t = ctx->rounds_enqueued + r, par = t & 1;
      launch_ex(ctx, ABS_KC_CTL, ctl_kernel, dim3(1), dim3(ctl_threads), csm, ctx->ctl, 1, 1, t, 0, 0);
      if (L.any_tc)
        launch_ex(ctx, ABS_KC_CTL, abs_times_kernel, dim3(times_blocks), dim3(32), 0, stc, ctx->ctl.job, ctx->ctl.next_dur, ctx->ctl.dur_job);
      q.ri = ctx->at<RoundInfo>(L.ri) + par;
      q.sel = ctx->ctl.sel[par]; q.sel_tau = ctx->ctl.sel_tau[par];
      q.row_idx = ctx->ctl.row_idx[par]; q.tile_slot = ctx->ctl.tile_slot[par];
      if (f32) launch_ex(ctx, ABS_KC_LSQ, lnet::local_begin_kernel<float>, dim3(bx, ctx->W), dim3(256), 0, q);
      else launch_ex(ctx, ABS_KC_LSQ, lnet::local_begin_kernel<__nv_bfloat16>, dim3(bx, ctx->W), dim3(256), 0, q);
      for (int u = 0; u < q.U; ++u) {
        gradient(par, PH_GATHER);
        gradient(par, PH_FORWARD);
        gradient(par, PH_BACKWARD);
        if (f32) launch_ex(ctx, ABS_KC_LSQ, lnet::local_step_kernel<float>, dim3(bx, ctx->W), dim3(256), 0, q, u);
        else launch_ex(ctx, ABS_KC_LSQ, lnet::local_step_kernel<__nv_bfloat16>, dim3(bx, ctx->W), dim3(256), 0, q, u);
      }
      update(par);
    }
    launch_ex(ctx, ABS_KC_CTL, ctl_kernel, dim3(1), dim3(ctl_threads), csm, ctx->ctl, 1, 0, ctx->rounds_enqueued + n, 0, 0);
  } else if (n > 0 && ctx->lsq_rounds) {
    LsqRoundsArgs q;
    q.X = ctx->X; q.y = (const float*)ctx->y;
    q.master = ctx->at<float>(ctx->L.master); q.ring = ctx->at<void>(ctx->L.ring);
    q.d_pad = ctx->L.d_pad; q.d = ctx->m.dims[0]; q.lr = ctx->m.lr;
    const size_t sm = lsq_rounds_smem(ctx->S, q.d);
    if (f32) launch_ex(ctx, ABS_KC_ROUNDS, abs_lsq_rounds_kernel<float>, dim3(1), dim3(LSQ_ROUNDS_NT), sm, ctx->ctl, q, ctx->rounds_enqueued, n);
    else launch_ex(ctx, ABS_KC_ROUNDS, abs_lsq_rounds_kernel<__nv_bfloat16>, dim3(1), dim3(LSQ_ROUNDS_NT), sm, ctx->ctl, q, ctx->rounds_enqueued, n);
  } else if (n > 0 && !ctx->overlap) {
    // One stream.  The control step of round t+1 does not depend on the Eq. 3 step of round t, which
    // is the kernel in front of it: it is launched without waiting for it (programmatic dependent
    // launch: it starts once every block of the Eq. 3 kernel has passed its own wait, i.e. once the
    // gradient kernels of round t are complete), runs next to it, prepares the next job durations
    // itself and waits for the Eq. 3 kernel at its end.  The first control step of a call follows
    // something else and waits at its start.
    for (int r = 0; r < n; ++r) {
      const int t = ctx->rounds_enqueued + r, par = t & 1;
      // the control kernel completes the previous round (if any) and selects this round's arrivals
      launch_ex(ctx, ABS_KC_CTL, ctl_kernel, dim3(1), dim3(ctl_threads), csm, ctx->ctl, 1, 1, t, r > 0 ? 1 : 0, 1);
      gradient(par, PH_GATHER);
      gradient(par, PH_FORWARD);
      gradient(par, PH_BACKWARD);
      update(par);
    }
    launch_ex(ctx, ABS_KC_CTL, ctl_kernel, dim3(1), dim3(ctl_threads), csm, ctx->ctl, 1, 0, ctx->rounds_enqueued + n, 1, 1);
  } else if (n > 0) {
    // Two streams.  Side stream per round t: control kernel (finish t-1, select t), row gather,
    // [event ctl], duration look-ahead.  Main stream: wait ctl, forward kernels, [event loss],
    // backward kernels and the Eq. 3 step.  The side stream's next control kernel waits for the
    // loss event only, so it overlaps the backward pass; layouts alternate by round parity.
    cudaStream_t A = ctx->stream, B = ctx->side;
    CU(cudaEventRecord(ctx->ev_loss, A));             // everything enqueued so far precedes the side work
    CU(cudaStreamWaitEvent(B, ctx->ev_loss, 0));
    for (int r = 0; r < n; ++r) {
      const int t = ctx->rounds_enqueued + r, par = t & 1;
      launch_on(ctx, B, ABS_KC_CTL, ctl_kernel, dim3(1), dim3(ctl_threads), csm, ctx->ctl, 1, 1, t, 0, 0);
      gradient(par, PH_GATHER);
      CU(cudaEventRecord(ctx->ev_ctl, B));
      launch_on(ctx, B, ABS_KC_CTL, abs_times_kernel, dim3(times_blocks), dim3(32), 0, stc, ctx->ctl.job, ctx->ctl.next_dur, ctx->ctl.dur_job);
      CU(cudaStreamWaitEvent(A, ctx->ev_ctl, 0));
      gradient(par, PH_FORWARD);
      CU(cudaEventRecord(ctx->ev_loss, A));
      CU(cudaStreamWaitEvent(B, ctx->ev_loss, 0));
      gradient(par, PH_BACKWARD);
      update(par);
    }
    launch_on(ctx, B, ABS_KC_CTL, ctl_kernel, dim3(1), dim3(ctl_threads), csm, ctx->ctl, 1, 0, ctx->rounds_enqueued + n, 0, 0);
    CU(cudaEventRecord(ctx->ev_ctl, B));
    CU(cudaStreamWaitEvent(A, ctx->ev_ctl, 0));       // the caller's stream covers all of it
  }
  if (ctx->launch_error != cudaSuccess) return cuda_fail(ctx, ctx->launch_error, "kernel launch");
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
  for (int b = 0; b < 2 && L.cnn; ++b)
    CU(cudaMemcpyAsync(dst + L.c_src[b], ctx->at<float>(L.master) + L.c_off[b], 4 * L.c_len[b], cudaMemcpyDeviceToHost, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  return ABS_OK;
}

namespace {

// Image of a context between rounds: header, then the two persistent regions of the workspace
// (control state .. ring, and the trace arrays).
struct StateHeader {
  unsigned long long magic;
  int version, rounds_enqueued;
  unsigned long long d_pad, esz, block1, block2, max_rounds;
  // what the saving context was created with (checked on restore)
  int kind, n_layers, dims[ABS_MAX_LAYERS + 1], conv[6], batch, dtype, local_steps, flags, restart_rule, sa_penalty;
  float lr;
  DevState st;                       // its state block (constants checked on restore)
};
constexpr unsigned long long STATE_MAGIC = 0x3230455441545341ull;   // "ASTATE02"

void describe_model(const abs_model_desc& m, StateHeader* h) {
  h->kind = m.kind; h->n_layers = m.n_layers;
  for (int l = 0; l <= ABS_MAX_LAYERS; ++l) h->dims[l] = l <= m.n_layers ? m.dims[l] : 0;
  for (int i = 0; i < 6; ++i) h->conv[i] = m.kind == ABS_CNN ? m.conv[i] : 0;
  h->batch = m.batch; h->dtype = m.dtype; h->local_steps = m.local_steps; h->flags = m.flags;
  h->restart_rule = m.restart_rule; h->sa_penalty = m.sa_penalty; h->lr = m.lr;
}

bool same_model(const StateHeader& a, const StateHeader& b) {
  bool same = a.kind == b.kind && a.n_layers == b.n_layers && a.batch == b.batch && a.dtype == b.dtype &&
              a.local_steps == b.local_steps && a.flags == b.flags && a.restart_rule == b.restart_rule &&
              a.sa_penalty == b.sa_penalty && a.lr == b.lr;
  for (int l = 0; l <= ABS_MAX_LAYERS; ++l) same = same && a.dims[l] == b.dims[l];
  for (int i = 0; i < 6; ++i) same = same && a.conv[i] == b.conv[i];
  return same;
}

void state_blocks(const Layout& L, size_t* b1_off, size_t* b1, size_t* b2_off, size_t* b2) {
  *b1_off = L.st;  *b1 = L.G - L.st;                           // control state, per-worker arrays, layouts, master, ring
  *b2_off = L.tr_K; *b2 = L.tr_rst_id - L.tr_K;                // trace arrays except the last ...
}

bool same_constants(const DevState& a, const DevState& b) {
  return a.W == b.W && a.K0 == b.K0 && a.S == b.S && a.B == b.B && a.RB == b.RB && a.k_mode == b.k_mode &&
         a.bound_mode == b.bound_mode && a.max_rounds == b.max_rounds && a.bound_offset == b.bound_offset &&
         a.theta_cap == b.theta_cap && a.literal_eq6 == b.literal_eq6 && a.no_restart == b.no_restart &&
         a.sa_penalty == b.sa_penalty && a.n_samples == b.n_samples &&
         a.key0 == b.key0 && a.key1 == b.key1 && a.dist.kind == b.dist.kind && a.dist.shift == b.dist.shift &&
         a.dist.rate == b.dist.rate && a.dist.scale == b.dist.scale && a.dist.slow_mod == b.dist.slow_mod &&
         a.dist.slow_rem == b.dist.slow_rem && a.dist.slow_factor == b.dist.slow_factor && a.dist.shape == b.dist.shape;
}

}  // namespace

int abs_state_bytes(abs_ctx* ctx, size_t* out) {
  if (!ctx || !out) return fail(ABS_EINVAL, "null argument");
  size_t o1, b1, o2, b2;
  state_blocks(ctx->L, &o1, &b1, &o2, &b2);
  b2 += 4 * (size_t)ctx->m.max_rounds * ctx->W;                // ... plus the last trace array (restarted ids)
  *out = sizeof(StateHeader) + b1 + b2;
  return ABS_OK;
}

int abs_save_state(abs_ctx* ctx, void* dst, size_t cap, size_t* written) {
  if (!ctx || !dst) return fail(ABS_EINVAL, "null argument");
  if (ctx->sticky != ABS_OK) return fail(ctx->sticky, "context is in a failed state (%d)", ctx->sticky);
  size_t total = 0;
  abs_state_bytes(ctx, &total);
  if (written) *written = total;
  if (cap < total) return fail(ABS_ENOSPACE, "destination holds %zu bytes, %zu needed", cap, total);
  size_t o1, b1, o2, b2;
  state_blocks(ctx->L, &o1, &b1, &o2, &b2);
  b2 += 4 * (size_t)ctx->m.max_rounds * ctx->W;
  StateHeader h;
  memset(&h, 0, sizeof h);
  int rc = read_status(ctx, &h.st);                            // synchronises the stream
  if (rc != ABS_OK) return rc;
  if (h.st.status != ST_OK) return fail(ABS_ESTATE, "the run has ended (status %d): nothing to continue from", h.st.status);
  if (h.st.open) return fail(ABS_ESTATE, "a round is open");
  h.magic = STATE_MAGIC; h.version = 2; h.rounds_enqueued = ctx->rounds_enqueued;
  describe_model(ctx->m, &h);
  h.d_pad = ctx->L.d_pad; h.esz = ctx->L.esz; h.block1 = b1; h.block2 = b2; h.max_rounds = (unsigned long long)ctx->m.max_rounds;
  char* p = (char*)dst;
  memcpy(p, &h, sizeof h);
  CU(cudaMemcpyAsync(p + sizeof h, ctx->ws + o1, b1, cudaMemcpyDeviceToHost, ctx->stream));
  CU(cudaMemcpyAsync(p + sizeof h + b1, ctx->ws + o2, b2, cudaMemcpyDeviceToHost, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  return ABS_OK;
}

int abs_restore_state(abs_ctx* ctx, const void* src, size_t bytes) {
  if (!ctx || !src) return fail(ABS_EINVAL, "null argument");
  if (ctx->sticky != ABS_OK) return fail(ctx->sticky, "context is in a failed state (%d)", ctx->sticky);
  if (bytes < sizeof(StateHeader)) return fail(ABS_EINVAL, "image shorter than its header");
  StateHeader h;
  memcpy(&h, src, sizeof h);
  if (h.magic != STATE_MAGIC || h.version != 2) return fail(ABS_EINVAL, "not a state image of this library version");
  StateHeader mine;
  memset(&mine, 0, sizeof mine);
  describe_model(ctx->m, &mine);
  if (!same_model(h, mine))
    return fail(ABS_EINVAL, "the image was saved by a context with another model, batch, step size, dtype, local steps, flags or modes");
  size_t o1, b1, o2, b2;
  state_blocks(ctx->L, &o1, &b1, &o2, &b2);
  b2 += 4 * (size_t)ctx->m.max_rounds * ctx->W;
  DevState cur;
  int rc = read_status(ctx, &cur);
  if (rc != ABS_OK) return rc;
  if (h.d_pad != ctx->L.d_pad || h.esz != ctx->L.esz || h.block1 != b1 || h.block2 != b2 ||
      h.max_rounds != (unsigned long long)ctx->m.max_rounds || !same_constants(h.st, cur))
    return fail(ABS_EINVAL, "the image was saved by a context with other sizes, modes, time distribution or seed");
  if (bytes != sizeof h + b1 + b2) return fail(ABS_EINVAL, "image has %zu bytes, %zu expected", bytes, sizeof h + b1 + b2);
  if (h.rounds_enqueued < 0 || h.rounds_enqueued > ctx->m.max_rounds || h.st.t != h.rounds_enqueued)
    return fail(ABS_EINVAL, "image is inconsistent (rounds %d, completed %d)", h.rounds_enqueued, h.st.t);
  const char* p = (const char*)src;
  CU(cudaMemcpyAsync(ctx->ws + o1, p + sizeof h, b1, cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaMemcpyAsync(ctx->ws + o2, p + sizeof h + b1, b2, cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  ctx->rounds_enqueued = h.rounds_enqueued;
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

int abs_get_plan(abs_ctx* ctx, int* partials, int* row_block, int* rows_cap, int* path) {
  if (!ctx) return fail(ABS_EINVAL, "ctx is null");
  if (partials) *partials = ctx->lsq_v2 ? ctx->lsq_grid : ctx->L.P;
  if (row_block) *row_block = ctx->L.RB;
  if (rows_cap) *rows_cap = ctx->L.rows_cap;
  if (path) for (int l = 0; l < ctx->m.n_layers; ++l) path[l] = ctx->L.path[l];
  return ABS_OK;
}

int abs_profile_start(abs_ctx* ctx, int max_launches) {
  if (!ctx || max_launches < 0) return fail(ABS_EINVAL, "bad argument");
  ctx->ev_class.clear();
  while ((int)ctx->ev.size() < 2 * max_launches) {
    cudaEvent_t e;
    CU(cudaEventCreate(&e));
    ctx->ev.push_back(e);
  }
  ctx->ev_cap = max_launches;
  return ABS_OK;
}

int abs_profile_read(abs_ctx* ctx, long long* launches, double* total_ms) {
  if (!ctx || !launches || !total_ms) return fail(ABS_EINVAL, "null argument");
  CU(cudaStreamSynchronize(ctx->stream));
  for (int c = 0; c < ABS_KC_COUNT; ++c) { launches[c] = 0; total_ms[c] = 0.0; }
  for (size_t i = 0; i < ctx->ev_class.size(); ++i) {
    float ms = 0.f;
    CU(cudaEventElapsedTime(&ms, ctx->ev[2 * i], ctx->ev[2 * i + 1]));
    launches[ctx->ev_class[i]] += 1;
    total_ms[ctx->ev_class[i]] += ms;
  }
  ctx->ev_cap = 0;
  ctx->ev_class.clear();
  return ABS_OK;
}

int abs_profile_timeline(abs_ctx* ctx, int cap, int* cls, float* start_ms, float* end_ms, int* n_out) {
  if (!ctx || !cls || !start_ms || !end_ms || !n_out || cap < 0) return fail(ABS_EINVAL, "bad argument");
  CU(cudaStreamSynchronize(ctx->stream));
  if (ctx->side) CU(cudaStreamSynchronize(ctx->side));
  const int n = std::min<int>(cap, (int)ctx->ev_class.size());
  for (int i = 0; i < n; ++i) {
    cls[i] = ctx->ev_class[i];
    CU(cudaEventElapsedTime(&start_ms[i], ctx->ev[0], ctx->ev[2 * i]));
    CU(cudaEventElapsedTime(&end_ms[i], ctx->ev[0], ctx->ev[2 * i + 1]));
  }
  *n_out = n;
  return ABS_OK;
}

int abs_selftest_wait_timeout(abs_ctx* ctx, int limit_us) {
  if (!ctx) return fail(ABS_EINVAL, "ctx is null");
  if (ctx->sticky != ABS_OK) return fail(ctx->sticky, "context is in a failed state (%d)", ctx->sticky);
  if (limit_us < 1 || limit_us > 1000000) return fail(ABS_EINVAL, "limit_us %d outside [1, 1000000]", limit_us);
  tc::wait_selftest_kernel<<<1, 32, 0, ctx->stream>>>(ctx->at<DevState>(ctx->L.st), 1000ull * (unsigned long long)limit_us);
  ctx->launches += 1;
  CU(cudaGetLastError());
  DevState h;
  const int rc = read_status(ctx, &h);
  if (rc != ABS_OK) return rc;
  return status_to_code(ctx, h);
}

int abs_destroy(abs_ctx* ctx) {
  if (!ctx) return ABS_OK;
  cudaStreamSynchronize(ctx->stream);
  for (cudaEvent_t e : ctx->ev) cudaEventDestroy(e);
  if (ctx->side) { cudaStreamSynchronize(ctx->side); cudaStreamDestroy(ctx->side); }
  if (ctx->ev_loss) cudaEventDestroy(ctx->ev_loss);
  if (ctx->ev_ctl) cudaEventDestroy(ctx->ev_ctl);
  delete ctx;
  return ABS_OK;
}

}  // extern "C"
