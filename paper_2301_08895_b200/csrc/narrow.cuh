// Memory-bound helpers around the hidden-layer GEMMs: minibatch row gather, the narrow output
// layer (at most 16 classes: forward + soft-max loss + delta in one pass, its back-propagation
// and its weight gradient) and bias gradients.  All are bound by HBM/L2 traffic, so they use
// plain coalesced loads and fixed-order reductions (bit-reproducible results).
#pragma once
#include "common.cuh"
#include "simt.cuh"

namespace absb {

constexpr int NARROW_MAX_C = 16;

// act0[r][:] = X[row_idx[r]][:] (zeros for padding rows); bf16, `in` a multiple of 8.
__global__ void __launch_bounds__(256) gather_rows_kernel(const DevState* st, const int* row_idx,
                                                          const __nv_bfloat16* X, __nv_bfloat16* act0, int in) {
  if (st->status != ST_OK) return;
  const int n_rows = st->n_rows;
  const int vec_per_row = in >> 3;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int r = blockIdx.x * 8 + warp; r < n_rows; r += gridDim.x * 8) {
    const int s = row_idx[r];
    uint4* dst = reinterpret_cast<uint4*>(act0 + (size_t)r * in);
    if (s < 0) {
      for (int v = lane; v < vec_per_row; v += 32) dst[v] = make_uint4(0u, 0u, 0u, 0u);
    } else {
      const uint4* src = reinterpret_cast<const uint4*>(X + (size_t)s * in);
      for (int v = lane; v < vec_per_row; v += 32) dst[v] = __ldg(src + v);
    }
  }
}

// Bias gradient of a hidden layer: G_p[b_off + n] = sum over the rows of chunk p of delta[r][n].
// Block = 32 column lanes x 32 row lanes; fixed-order reduction.
template <typename T>
__global__ void __launch_bounds__(1024) colsum_kernel(const DevState* st, const T* delta, float* G, size_t slot_stride,
                                                      size_t b_off, int out, int P) {
  __shared__ float red[32][33];
  if (st->status != ST_OK) return;
  const int n_rows = st->n_rows;
  const int chunk = round_up((n_rows + P - 1) / P, 64);
  const int p = blockIdx.y;
  const int k_begin = min(n_rows, p * chunk), k_end = min(n_rows, (p + 1) * chunk);
  const int cl = threadIdx.x & 31, rl = threadIdx.x >> 5;
  const int n = blockIdx.x * 32 + cl;
  float acc = 0.f;
  if (n < out)
    for (int r = k_begin + rl; r < k_end; r += 32) acc += ldf(delta, (size_t)r * out + n);
  red[rl][cl] = acc;
  __syncthreads();
  if (rl == 0 && n < out) {
    float tot = 0.f;
    for (int q = 0; q < 32; ++q) tot += red[q][cl];
    G[(size_t)p * slot_stride + b_off + n] = tot;
  }
}

struct NarrowArgs {
  DevState* st;
  const int* tile_slot;
  const int* row_idx;
  const int* labels;
  const void* ring; size_t slot_stride; size_t w_off;
  int in, C;
  int gather;              // input rows come from X[row_idx[r]] (soft-max regression)
  const void* act_in;      // [rows][in] or X
  void* delta_out;         // [rows][C] storage type
  void* delta_in;          // [rows][in] storage type (dgrad result)
  float* row_loss;         // [rows]
  float* G; int P;
};

// Output layer forward + soft-max cross-entropy + delta for 64 rows per block (one ring slot).
// One warp per row: lanes stride over the input features, C accumulators each.
template <typename T>
__global__ void __launch_bounds__(256) narrow_fwd_loss_kernel(NarrowArgs a) {
  extern __shared__ float wsm[];               // [in][C] then bias[C]
  DevState* st = a.st;
  if (st->status != ST_OK) return;
  const int r0 = blockIdx.x * 64;
  if (r0 >= st->n_rows) return;
  const int in = a.in, C = a.C;
  const int slot = a.tile_slot[r0 / st->RB];
  const T* Wm = (const T*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
  for (int i = threadIdx.x; i < in * C + C; i += 256) wsm[i] = ldf(Wm, i);
  __syncthreads();
  const float* bias = wsm + (size_t)in * C;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const T* src = (const T*)a.act_in;
  bool bad = false;
  for (int rr = warp; rr < 64; rr += 8) {
    const int r = r0 + rr;
    const int s = a.row_idx[r];
    T* d = (T*)a.delta_out + (size_t)r * C;
    if (s < 0) {                               // padding row: contributes nothing to Eq. 3
      if (lane < C) stf(d, lane, 0.f);
      if (lane == 0) a.row_loss[r] = 0.f;
      continue;
    }
    const T* x = a.gather ? src + (size_t)s * in : src + (size_t)r * in;
    float acc[NARROW_MAX_C];
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c) acc[c] = 0.f;
    for (int k = lane; k < in; k += 32) {
      const float xv = ldf(x, k);
      const float* wr = wsm + (size_t)k * C;
#pragma unroll
      for (int c = 0; c < NARROW_MAX_C; ++c)
        if (c < C) acc[c] = fmaf(xv, wr[c], acc[c]);
    }
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c)
      if (c < C) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], o);
        acc[c] += bias[c];
      }
    const int y = a.labels[s];
    float zmax = acc[0], zy = 0.f;
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c)
      if (c < C) { zmax = fmaxf(zmax, acc[c]); if (c == y) zy = acc[c]; }
    float se = 0.f;
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c)
      if (c < C) { acc[c] = expf(acc[c] - zmax); se += acc[c]; }
    const float inv = 1.f / se;
    float mine = 0.f;
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c)
      if (c == lane) mine = acc[c] * inv - (c == y ? 1.f : 0.f);
    if (lane < C) stf(d, lane, mine);
    const float loss = logf(se) - (zy - zmax);
    if (lane == 0) a.row_loss[r] = loss;
    bad |= !isfinite(loss);
  }
  if (bad && lane == 0) st->diverged = 1;
}

// Back-propagation through the output layer and the ReLU before it, 64 rows per block:
// delta_in[r][m] = (sum_c delta_out[r][c] W_s[m][c]) * [act_in[r][m] > 0].
template <typename T>
__global__ void __launch_bounds__(256) narrow_dgrad_kernel(NarrowArgs a) {
  extern __shared__ float wsm[];               // [in][C] then delta tile [64][C]
  DevState* st = a.st;
  if (st->status != ST_OK) return;
  const int r0 = blockIdx.x * 64;
  if (r0 >= st->n_rows) return;
  const int in = a.in, C = a.C;
  const int slot = a.tile_slot[r0 / st->RB];
  const T* Wm = (const T*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
  float* dsm = wsm + (size_t)in * C;
  for (int i = threadIdx.x; i < in * C; i += 256) wsm[i] = ldf(Wm, i);
  const T* dl = (const T*)a.delta_out + (size_t)r0 * C;
  for (int i = threadIdx.x; i < 64 * C; i += 256) dsm[i] = ldf(dl, i);
  __syncthreads();
  const T* h = (const T*)a.act_in;
  T* out = (T*)a.delta_in;
  for (int m = threadIdx.x; m < in; m += 256) {
    float w[NARROW_MAX_C];
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c) w[c] = (c < C) ? wsm[(size_t)m * C + c] : 0.f;
    for (int rr = 0; rr < 64; ++rr) {
      float acc = 0.f;
#pragma unroll
      for (int c = 0; c < NARROW_MAX_C; ++c)
        if (c < C) acc = fmaf(dsm[rr * C + c], w[c], acc);
      const size_t o = (size_t)(r0 + rr) * in + m;
      stf(out, o, ldf(h, o) > 0.f ? acc : 0.f);
    }
  }
}

// Weight and bias gradient of the output layer over the rows of chunk p:
// G_p[m][c] = sum_r act_in[r][m] delta_out[r][c], row m = `in` is the bias gradient.
// Block = 32 feature lanes x 32 row lanes, fixed-order reduction over the row lanes.
template <typename T>
__global__ void __launch_bounds__(1024) narrow_wgrad_kernel(NarrowArgs a) {
  __shared__ float red[32][33];
  DevState* st = a.st;
  if (st->status != ST_OK) return;
  const int in = a.in, C = a.C;
  const int n_rows = st->n_rows;
  const int chunk = round_up((n_rows + a.P - 1) / a.P, 64);
  const int p = blockIdx.y;
  const int k_begin = min(n_rows, p * chunk), k_end = min(n_rows, (p + 1) * chunk);
  const int ml = threadIdx.x & 31, rl = threadIdx.x >> 5;
  const int m = blockIdx.x * 32 + ml;
  const T* src = (const T*)a.act_in;
  const T* dl = (const T*)a.delta_out;
  float acc[NARROW_MAX_C];
#pragma unroll
  for (int c = 0; c < NARROW_MAX_C; ++c) acc[c] = 0.f;
  if (m <= in) {
    for (int r = k_begin + rl; r < k_end; r += 32) {
      float xv;
      if (m == in) xv = 1.f;
      else if (a.gather) {
        const int s = a.row_idx[r];
        xv = s < 0 ? 0.f : ldf(src, (size_t)s * in + m);
      } else xv = ldf(src, (size_t)r * in + m);
#pragma unroll
      for (int c = 0; c < NARROW_MAX_C; ++c)
        if (c < C) acc[c] = fmaf(xv, ldf(dl, (size_t)r * C + c), acc[c]);
    }
  }
  float* G = a.G + (size_t)p * a.slot_stride + a.w_off;
#pragma unroll
  for (int c = 0; c < NARROW_MAX_C; ++c) {
    if (c < C) {                                // C is uniform across the block
      red[rl][ml] = acc[c];
      __syncthreads();
      if (rl == 0 && m <= in) {
        float tot = 0.f;
        for (int q = 0; q < 32; ++q) tot += red[q][ml];
        G[(size_t)m * C + c] = tot;
      }
      __syncthreads();
    }
  }
}

}  // namespace absb
