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
__global__ void __launch_bounds__(256) gather_rows_kernel(const DevState* st, const RoundInfo* ri, const int* row_idx,
                                                          const __nv_bfloat16* X, __nv_bfloat16* act0, int in) {
  grid_dependency_sync();
  if (st->status != ST_OK) return;
  const int n_rows = ri->n_rows;
  const int vec_per_row = in >> 3;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int r = blockIdx.x * 8 + warp; r < n_rows; r += gridDim.x * 8) {
    const int s = row_idx[r];
    uint4* dst = reinterpret_cast<uint4*>(act0 + (size_t)r * in);
    if (s < 0) {
      for (int v = lane; v < vec_per_row; v += 32) dst[v] = make_uint4(0u, 0u, 0u, 0u);
    } else {
      // four 16-byte loads per lane in flight before the first store
      const uint4* src = reinterpret_cast<const uint4*>(X + (size_t)s * in);
      for (int v = lane; v < vec_per_row; v += 128) {
        uint4 q[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (v + 32 * k < vec_per_row) q[k] = __ldg(src + v + 32 * k);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (v + 32 * k < vec_per_row) dst[v + 32 * k] = q[k];
      }
    }
  }
}

struct NarrowArgs {
  DevState* st;
  RoundInfo* ri;
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
  int rpb;                 // gradient rows per block of the row-tiled kernels below (8..64, a multiple of 8; 0 = 64)
};

// Output layer forward + soft-max cross-entropy + delta for 64 rows per block (one ring slot).
// One warp per row: lanes stride over the input features, C accumulators each.
template <typename T>
__global__ void __launch_bounds__(256) narrow_fwd_loss_kernel(NarrowArgs a) {
  grid_dependency_sync();
  extern __shared__ float wsm[];               // [in][C] then bias[C]
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int RPB = a.rpb ? a.rpb : 64;
  const int r0 = blockIdx.x * RPB;
  if (r0 >= ri->n_rows) return;
  const int in = a.in, C = a.C;
  const int slot = a.tile_slot[r0 / st->RB];
  const float sa = sa_slot_weight(st, ri->t, slot);     // staleness-aware step size: weight of these rows in Eq. 3
  const T* Wm = (const T*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
  for (int i = threadIdx.x; i < in * C + C; i += 256) wsm[i] = ldf(Wm, i);
  __syncthreads();
  const float* bias = wsm + (size_t)in * C;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const T* src = (const T*)a.act_in;
  bool bad = false;
  for (int rr = warp; rr < RPB; rr += 8) {
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
      if (c == lane) mine = (acc[c] * inv - (c == y ? 1.f : 0.f)) * sa;
    if (lane < C) stf(d, lane, mine);
    const float loss = logf(se) - (zy - zmax);
    if (lane == 0) a.row_loss[r] = loss;
    bad |= !isfinite(loss);
  }
  if (bad && lane == 0) ri->diverged = 1;
}

// Back-propagation through the output layer and the ReLU before it, 64 rows per block:
// delta_in[r][m] = (sum_c delta_out[r][c] W_s[m][c]) * [act_in[r][m] > 0].
template <typename T>
__global__ void __launch_bounds__(256) narrow_dgrad_kernel(NarrowArgs a) {
  grid_dependency_sync();
  extern __shared__ float wsm[];               // [in][C] then delta tile [64][C]
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int RPB = a.rpb ? a.rpb : 64;
  const int r0 = blockIdx.x * RPB;
  if (r0 >= ri->n_rows) return;
  const int in = a.in, C = a.C;
  const int slot = a.tile_slot[r0 / st->RB];
  const T* Wm = (const T*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
  float* dsm = wsm + (size_t)in * C;
  for (int i = threadIdx.x; i < in * C; i += 256) wsm[i] = ldf(Wm, i);
  const T* dl = (const T*)a.delta_out + (size_t)r0 * C;
  for (int i = threadIdx.x; i < RPB * C; i += 256) dsm[i] = ldf(dl, i);
  __syncthreads();
  const T* h = (const T*)a.act_in;
  T* out = (T*)a.delta_in;
  for (int m = threadIdx.x; m < in; m += 256) {
    float w[NARROW_MAX_C];
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c) w[c] = (c < C) ? wsm[(size_t)m * C + c] : 0.f;
    for (int rr = 0; rr < RPB; ++rr) {
      float acc = 0.f;
#pragma unroll
      for (int c = 0; c < NARROW_MAX_C; ++c)
        if (c < C) acc = fmaf(dsm[rr * C + c], w[c], acc);
      const size_t o = (size_t)(r0 + rr) * in + m;
      stf(out, o, ldf(h, o) > 0.f ? acc : 0.f);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Vectorised variants (feature counts that are multiples of 8): 16-byte loads, weights kept in
// shared memory transposed ([class][feature], storage type) so that a lane's 8 consecutive
// features of one class are one conflict-free 16-byte read.

__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 u = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int j = 0; j < 4; ++j) { const float2 f = __bfloat1622float2(h[j]); v[2 * j] = f.x; v[2 * j + 1] = f.y; }
}
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
  const float4 a = reinterpret_cast<const float4*>(p)[0], b = reinterpret_cast<const float4*>(p)[1];
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void store8(__nv_bfloat16* p, const float (&v)[8]) {
  uint4 u;
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&u);
#pragma unroll
  for (int j = 0; j < 4; ++j) h[j] = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
  *reinterpret_cast<uint4*>(p) = u;
}
__device__ __forceinline__ void store8(float* p, const float (&v)[8]) {
  reinterpret_cast<float4*>(p)[0] = make_float4(v[0], v[1], v[2], v[3]);
  reinterpret_cast<float4*>(p)[1] = make_float4(v[4], v[5], v[6], v[7]);
}

constexpr int NARROW_ROWS = 16;   // rows per block of the vectorised forward / dgrad kernels

// Output layer forward + soft-max cross-entropy + delta, 16 rows per block, one warp per row pair.
template <typename T>
__global__ void __launch_bounds__(256) narrow_fwd_loss_v8_kernel(NarrowArgs a) {
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char nsm_raw[];
  T* wT = reinterpret_cast<T*>(nsm_raw);                 // [C][in]
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int r0 = blockIdx.x * NARROW_ROWS;
  if (r0 >= ri->n_rows) return;
  const int in = a.in, C = a.C;
  float* bias = reinterpret_cast<float*>(wT + (size_t)C * in);
  const int slot = a.tile_slot[r0 / st->RB];
  const float sa = sa_slot_weight(st, ri->t, slot);     // staleness-aware step size: weight of these rows in Eq. 3
  const T* Wm = (const T*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
#pragma unroll 8
  for (int i = threadIdx.x; i < in * C; i += 256) {
    const int k = i / C, c = i - k * C;
    wT[(size_t)c * in + k] = Wm[i];
  }
  if (threadIdx.x < C) bias[threadIdx.x] = ldf(Wm, (size_t)in * C + threadIdx.x);
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const T* src = (const T*)a.act_in;
  const int nvec = in >> 3;
  bool bad = false;
  for (int rr = warp; rr < NARROW_ROWS; rr += 8) {
    const int r = r0 + rr;
    const int s = a.row_idx[r];
    T* d = (T*)a.delta_out + (size_t)r * C;
    if (s < 0) {
      if (lane < C) stf(d, lane, 0.f);
      if (lane == 0) a.row_loss[r] = 0.f;
      continue;
    }
    const T* x = a.gather ? src + (size_t)s * in : src + (size_t)r * in;
    float acc[NARROW_MAX_C];
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c) acc[c] = 0.f;
#pragma unroll 2
    for (int v = lane; v < nvec; v += 32) {
      float xv[8];
      load8(x + v * 8, xv);
#pragma unroll
      for (int c = 0; c < NARROW_MAX_C; ++c)
        if (c < C) {
          float wv[8];
          load8(wT + (size_t)c * in + v * 8, wv);
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[c] = fmaf(xv[j], wv[j], acc[c]);
        }
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
      if (c == lane) mine = (acc[c] * inv - (c == y ? 1.f : 0.f)) * sa;
    if (lane < C) stf(d, lane, mine);
    const float loss = logf(se) - (zy - zmax);
    if (lane == 0) a.row_loss[r] = loss;
    bad |= !isfinite(loss);
  }
  if (bad && lane == 0) ri->diverged = 1;
}

// Back-propagation through the output layer and the ReLU before it, 16 rows per block; a work
// item is (row, 8 consecutive features).
template <typename T>
__global__ void __launch_bounds__(256) narrow_dgrad_v8_kernel(NarrowArgs a) {
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char nsm_raw[];
  T* wT = reinterpret_cast<T*>(nsm_raw);                 // [C][in]
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int r0 = blockIdx.x * NARROW_ROWS;
  if (r0 >= ri->n_rows) return;
  const int in = a.in, C = a.C;
  float* dsm = reinterpret_cast<float*>(wT + (size_t)C * in);   // [16][C]
  const int slot = a.tile_slot[r0 / st->RB];
  const T* Wm = (const T*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
#pragma unroll 8
  for (int i = threadIdx.x; i < in * C; i += 256) {
    const int k = i / C, c = i - k * C;
    wT[(size_t)c * in + k] = Wm[i];
  }
  const T* dl = (const T*)a.delta_out + (size_t)r0 * C;
  for (int i = threadIdx.x; i < NARROW_ROWS * C; i += 256) dsm[i] = ldf(dl, i);
  __syncthreads();
  const T* h = (const T*)a.act_in;
  T* out = (T*)a.delta_in;
  const int nvec = in >> 3;
  for (int item = threadIdx.x; item < NARROW_ROWS * nvec; item += 256) {
    const int rr = item / nvec, v = item - rr * nvec;
    const size_t o = (size_t)(r0 + rr) * in + (size_t)v * 8;
    float hv[8], acc[8];
    load8(h + o, hv);
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.f;
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c)
      if (c < C) {
        float wv[8];
        load8(wT + (size_t)c * in + v * 8, wv);
        const float dv = dsm[rr * C + c];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = fmaf(dv, wv[j], acc[j]);
      }
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = hv[j] > 0.f ? acc[j] : 0.f;
    store8(out + o, acc);
  }
}

__device__ __forceinline__ void load2(const __nv_bfloat16* p, float& x, float& y) {
  const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p));
  x = f.x; y = f.y;
}
__device__ __forceinline__ void load2(const float* p, float& x, float& y) {
  const float2 f = *reinterpret_cast<const float2*>(p);
  x = f.x; y = f.y;
}

// Stage 1 of the output layer's weight gradient: per 64-row chunk q,
// part[q][m][c] = sum_{r in chunk} act_in[r][m] delta_out[r][c], with row m = `in` the bias sums.
// A thread owns two neighbouring features (one 4/8-byte load per row), rows are fetched eight
// at a time so the loads overlap.  Padding rows have zero deltas, so whatever finite input they
// point at adds nothing.
template <typename T>
__global__ void __launch_bounds__(256) narrow_wgrad_chunk_kernel(NarrowArgs a, float* part) {
  grid_dependency_sync();
  __shared__ float dsm[64][NARROW_MAX_C];
  __shared__ long long rowoff[64];
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int RPB = a.rpb ? a.rpb : 64;
  const int r0 = blockIdx.x * RPB;
  if (r0 >= ri->n_rows) return;
  const int in = a.in, C = a.C;
  const T* dl = (const T*)a.delta_out + (size_t)r0 * C;
  for (int i = threadIdx.x; i < RPB * C; i += 256) dsm[i / C][i % C] = ldf(dl, i);
  if (threadIdx.x < RPB) {
    const int r = r0 + threadIdx.x;
    long long off = (long long)r * in;
    if (a.gather) { const int s = a.row_idx[r]; off = s < 0 ? 0 : (long long)s * in; }
    rowoff[threadIdx.x] = off;
  }
  __syncthreads();
  const T* src = (const T*)a.act_in;
  float* dst = part + (size_t)blockIdx.x * (size_t)(in + 1) * C;
  const bool pairs = (in & 1) == 0;
  const int n_items = pairs ? in / 2 : in;
  for (int it = threadIdx.x; it < n_items; it += 256) {
    const int m = pairs ? 2 * it : it;
    float acc0[NARROW_MAX_C], acc1[NARROW_MAX_C];
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c) { acc0[c] = 0.f; acc1[c] = 0.f; }
    for (int rb = 0; rb < RPB; rb += 8) {
      float x0[8], x1[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const T* px = src + (size_t)rowoff[rb + j] + m;
        if (pairs) load2(px, x0[j], x1[j]);
        else { x0[j] = ldf(px, 0); x1[j] = 0.f; }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int c = 0; c < NARROW_MAX_C; ++c)
          if (c < C) {
            const float dv = dsm[rb + j][c];
            acc0[c] = fmaf(x0[j], dv, acc0[c]);
            acc1[c] = fmaf(x1[j], dv, acc1[c]);
          }
    }
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c)
      if (c < C) {
        dst[(size_t)m * C + c] = acc0[c];
        if (pairs) dst[(size_t)(m + 1) * C + c] = acc1[c];
      }
  }
  if (threadIdx.x < C) {                       // bias row: column sums of the deltas
    float tot = 0.f;
    for (int rr = 0; rr < RPB; ++rr) tot += dsm[rr][threadIdx.x];
    dst[(size_t)in * C + threadIdx.x] = tot;
  }
}

// Stage 2: dst[i] = sum over the active chunks q of part[q][i], i < len.  Block = 32 outputs x 8
// chunk lanes; lane w adds chunks w, w+8, ... in order, then the 8 lanes are added in order.
__global__ void __launch_bounds__(256) chunk_reduce_kernel(const DevState* st, const RoundInfo* ri, const float* part, int len, float* dst,
                                                           int chunk_rows) {
  grid_dependency_sync();
  __shared__ float red[8][33];
  if (st->status != ST_OK) return;
  const int n_chunks = ri->n_rows / chunk_rows;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int i = blockIdx.x * 32 + lane;
  float acc = 0.f;
  if (i < len) {
#pragma unroll 8
    for (int q = w; q < n_chunks; q += 8) acc += part[(size_t)q * len + i];
  }
  red[w][lane] = acc;
  __syncthreads();
  if (w == 0 && i < len) {
    float tot = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) tot += red[q][lane];
    dst[i] = tot;
  }
}

__device__ __forceinline__ void copy8(__nv_bfloat16* dst, const __nv_bfloat16* src) {
  *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
}
__device__ __forceinline__ void copy8(float* dst, const float* src) {
  reinterpret_cast<float4*>(dst)[0] = reinterpret_cast<const float4*>(src)[0];
  reinterpret_cast<float4*>(dst)[1] = reinterpret_cast<const float4*>(src)[1];
}
__device__ __forceinline__ void zero8(__nv_bfloat16* dst) { *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u); }
__device__ __forceinline__ void zero8(float* dst) {
  reinterpret_cast<float4*>(dst)[0] = make_float4(0.f, 0.f, 0.f, 0.f);
  reinterpret_cast<float4*>(dst)[1] = make_float4(0.f, 0.f, 0.f, 0.f);
}
__device__ __forceinline__ float round_store(float x, const __nv_bfloat16*) { return __bfloat162float(__float2bfloat16_rn(x)); }
__device__ __forceinline__ float round_store(float x, const float*) { return x; }

// The whole output layer in one pass over R rows per block (R rows of the layer's input stay in
// shared memory): logits, soft-max cross-entropy loss and delta (Eq. 2 at the rows' model
// version), the back-propagated delta of the layer below, and this block's share of the layer's
// weight and bias gradient (part[block][m][c], row m = `in` the bias sums; stage 2 adds the blocks
// up in order).  Feature count a multiple of 8, at most 16 classes.
template <typename T>
__global__ void __launch_bounds__(256) narrow_fused_kernel(NarrowArgs a, float* part, int R, int has_dgrad) {
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char nsm_raw[];
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int r0 = blockIdx.x * R;
  if (r0 >= ri->n_rows) return;
  const int in = a.in, C = a.C, nvec = in >> 3;
  const int wld = in + 8;                                      // padded row of the transposed weights
  T* hs = reinterpret_cast<T*>(nsm_raw);                       // [R][in] input rows
  T* wT = hs + (size_t)R * in;                                 // [C][in + 8] weights, transposed
  T* wraw = wT + (size_t)C * wld;                              // [in][C] + bias[C] as stored
  float* d3 = reinterpret_cast<float*>(wraw + (size_t)(in + 1) * C + 8);  // [R][16] deltas of this layer's output
  d3 = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(d3) + 15) & ~(uintptr_t)15);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const T* src = (const T*)a.act_in;
  // asynchronous 16-byte copies: every thread issues all of its copies before anyone waits
  constexpr int PIECES = sizeof(T) * 8 / 16;                   // 16-byte pieces per 8 elements
  for (int item = tid; item < R * nvec; item += 256) {
    const int rr = item / nvec, v = item - rr * nvec;
    long long row = r0 + rr;
    if (a.gather) row = a.row_idx[r0 + rr];
    T* d = hs + (size_t)rr * in + v * 8;
    if (row < 0) zero8(d);
    else {
      const T* g = src + (size_t)row * in + v * 8;
#pragma unroll
      for (int q = 0; q < PIECES; ++q)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(
                         reinterpret_cast<unsigned char*>(d) + 16 * q)), "l"(reinterpret_cast<const unsigned char*>(g) + 16 * q) : "memory");
    }
  }
  const int slot = a.tile_slot[r0 / st->RB];
  const float sa = sa_slot_weight(st, ri->t, slot);     // staleness-aware step size: weight of these rows in Eq. 3
  const T* Wm = (const T*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
  {
    // weights + bias are contiguous and start on a 128-byte boundary; copy whole 16-byte pieces
    const int n16 = (int)(((size_t)(in + 1) * C * sizeof(T) + 15) / 16);
    for (int i = tid; i < n16; i += 256)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(
                       reinterpret_cast<unsigned char*>(wraw) + 16 * i)), "l"(reinterpret_cast<const unsigned char*>(Wm) + 16 * i) : "memory");
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  for (int i = tid; i < in * C; i += 256) {
    const int k = i / C, c = i - k * C;
    wT[(size_t)c * wld + k] = wraw[i];
  }
  const T* bias = wraw + (size_t)in * C;
  __syncthreads();
  // ---- logits, loss, delta: one warp per row
  bool bad = false;
  for (int rr = warp; rr < R; rr += 8) {
    const int r = r0 + rr;
    const int s = a.row_idx[r];
    if (s < 0) {                                // padding row: contributes nothing to Eq. 3
      if (lane < NARROW_MAX_C) d3[rr * NARROW_MAX_C + lane] = 0.f;
      if (lane == 0) a.row_loss[r] = 0.f;
      continue;
    }
    const T* x = hs + (size_t)rr * in;
    float acc[NARROW_MAX_C];
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c) acc[c] = 0.f;
    for (int v = lane; v < nvec; v += 32) {
      float xv[8];
      load8(x + v * 8, xv);
#pragma unroll
      for (int c = 0; c < NARROW_MAX_C; ++c)
        if (c < C) {
          float wv[8];
          load8(wT + (size_t)c * wld + v * 8, wv);
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[c] = fmaf(xv[j], wv[j], acc[c]);
        }
    }
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c)
      if (c < C) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], o);
        acc[c] += ldf(bias, c);
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
      if (c == lane) mine = (acc[c] * inv - (c == y ? 1.f : 0.f)) * sa;
    // the delta is a stored quantity: round it to the storage type like every other delta
    if (lane < NARROW_MAX_C) d3[rr * NARROW_MAX_C + lane] = lane < C ? round_store(mine, (const T*)nullptr) : 0.f;
    const float loss = logf(se) - (zy - zmax);
    if (lane == 0) a.row_loss[r] = loss;
    bad |= !isfinite(loss);
  }
  if (bad && lane == 0) ri->diverged = 1;
  __syncthreads();
  // ---- delta of the layer below: (delta W^T) masked by the ReLU of the input rows
  if (has_dgrad) {
    T* out = (T*)a.delta_in;
    for (int item = tid; item < R * nvec; item += 256) {
      const int rr = item / nvec, v = item - rr * nvec;
      float hv[8], acc[8];
      load8(hs + (size_t)rr * in + v * 8, hv);
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = 0.f;
#pragma unroll
      for (int c = 0; c < NARROW_MAX_C; ++c)
        if (c < C) {
          float wv[8];
          load8(wT + (size_t)c * wld + v * 8, wv);
          const float dv = d3[rr * NARROW_MAX_C + c];
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[j] = fmaf(dv, wv[j], acc[j]);
        }
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = hv[j] > 0.f ? acc[j] : 0.f;
      store8(out + (size_t)(r0 + rr) * in + (size_t)v * 8, acc);
    }
  }
  // ---- this block's share of the weight and bias gradient
  float* dst = part + (size_t)blockIdx.x * (size_t)(in + 1) * C;
  for (int it = tid; it < in / 2; it += 256) {
    const int m = 2 * it;
    float acc0[NARROW_MAX_C], acc1[NARROW_MAX_C];
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c) { acc0[c] = 0.f; acc1[c] = 0.f; }
    for (int rr = 0; rr < R; ++rr) {
      float x0, x1;
      load2(hs + (size_t)rr * in + m, x0, x1);
#pragma unroll
      for (int c = 0; c < NARROW_MAX_C; ++c)
        if (c < C) {
          const float dv = d3[rr * NARROW_MAX_C + c];
          acc0[c] = fmaf(x0, dv, acc0[c]);
          acc1[c] = fmaf(x1, dv, acc1[c]);
        }
    }
#pragma unroll
    for (int c = 0; c < NARROW_MAX_C; ++c)
      if (c < C) { dst[(size_t)m * C + c] = acc0[c]; dst[(size_t)(m + 1) * C + c] = acc1[c]; }
  }
  if (tid < C) {
    float tot = 0.f;
    for (int rr = 0; rr < R; ++rr) tot += d3[rr * NARROW_MAX_C + tid];
    dst[(size_t)in * C + tid] = tot;
  }
}

// Same operation as narrow_fused_kernel with the class count CC known at compile time: weights are
// kept as fp32 in shared memory, every weight fetched from shared memory is used for four rows
// (forward) or stays in registers for all rows of the block (delta of the layer below).
template <typename T, int CC>
__global__ void __launch_bounds__(256) narrow_fused_cc_kernel(NarrowArgs a, float* part, int R, int has_dgrad) {
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char nsm_raw[];
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int r0 = blockIdx.x * R;
  if (r0 >= ri->n_rows) return;
  const int in = a.in, nvec = in >> 3;
  const int wld = in + 4;                                      // padded row of the transposed fp32 weights
  T* hs = reinterpret_cast<T*>(nsm_raw);                       // [R][in] input rows
  float* wf = reinterpret_cast<float*>(hs + (size_t)R * in);   // [CC][in + 4]
  float* d3 = wf + (size_t)CC * wld;                           // [R][CC] deltas of this layer's output
  T* wraw = reinterpret_cast<T*>(d3 + (size_t)R * CC);         // [in][CC] + bias[CC] as stored (16-byte aligned)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const T* src = (const T*)a.act_in;
  constexpr int PIECES = sizeof(T) * 8 / 16;
  for (int item = tid; item < R * nvec; item += 256) {
    const int rr = item / nvec, v = item - rr * nvec;
    long long row = r0 + rr;
    if (a.gather) row = a.row_idx[r0 + rr];
    T* d = hs + (size_t)rr * in + v * 8;
    if (row < 0) zero8(d);
    else {
      const T* g = src + (size_t)row * in + v * 8;
#pragma unroll
      for (int q = 0; q < PIECES; ++q)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(
                         reinterpret_cast<unsigned char*>(d) + 16 * q)), "l"(reinterpret_cast<const unsigned char*>(g) + 16 * q) : "memory");
    }
  }
  const int slot = a.tile_slot[r0 / st->RB];
  const float sa = sa_slot_weight(st, ri->t, slot);     // staleness-aware step size: weight of these rows in Eq. 3
  const T* Wm = (const T*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
  {
    const int n16 = (int)(((size_t)(in + 1) * CC * sizeof(T) + 15) / 16);
    for (int i = tid; i < n16; i += 256)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(
                       reinterpret_cast<unsigned char*>(wraw) + 16 * i)), "l"(reinterpret_cast<const unsigned char*>(Wm) + 16 * i) : "memory");
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  for (int i = tid; i < in * CC; i += 256) {
    const int k = i / CC, c = i - k * CC;
    wf[(size_t)c * wld + k] = ldf(wraw, i);
  }
  __syncthreads();
  // ---- logits, loss, delta: a warp takes four rows at a time (two, one when the block has fewer
  // rows than that keeps all eight warps busy; a row's sum is formed in the same order either way)
  bool bad = false;
  const int rpw = R >= 32 ? 4 : (R >= 16 ? 2 : 1);
  for (int rb = warp * rpw; rb < R; rb += 8 * rpw) {
    float acc[4][CC];
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
      for (int c = 0; c < CC; ++c) acc[q][c] = 0.f;
    for (int v = lane; v < nvec; v += 32) {
      float xv[4][8];
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (q < rpw) load8(hs + (size_t)(rb + q) * in + v * 8, xv[q]);
#pragma unroll
      for (int c = 0; c < CC; ++c) {
        float wv[8];
        load8(wf + (size_t)c * wld + v * 8, wv);
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (q < rpw) {
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[q][c] = fmaf(xv[q][j], wv[j], acc[q][c]);
          }
      }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (q < rpw) {
#pragma unroll
        for (int c = 0; c < CC; ++c)
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) acc[q][c] += __shfl_xor_sync(0xffffffffu, acc[q][c], o);
      }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (q >= rpw) break;
      const int rr = rb + q, r = r0 + rr;
      const int s = a.row_idx[r];
      if (s < 0) {                              // padding row: contributes nothing to Eq. 3
        if (lane < CC) d3[rr * CC + lane] = 0.f;
        if (lane == 0) a.row_loss[r] = 0.f;
        continue;
      }
      const int y = a.labels[s];
      float z[CC];
      float zmax = -3.0e38f, zy = 0.f;
#pragma unroll
      for (int c = 0; c < CC; ++c) {
        z[c] = acc[q][c] + ldf(wraw, (size_t)in * CC + c);
        zmax = fmaxf(zmax, z[c]);
        if (c == y) zy = z[c];
      }
      float se = 0.f;
#pragma unroll
      for (int c = 0; c < CC; ++c) { z[c] = expf(z[c] - zmax); se += z[c]; }
      const float inv = 1.f / se;
      float mine = 0.f;
#pragma unroll
      for (int c = 0; c < CC; ++c)
        if (c == lane) mine = (z[c] * inv - (c == y ? 1.f : 0.f)) * sa;
      // the delta is a stored quantity: round it to the storage type like every other delta
      if (lane < CC) d3[rr * CC + lane] = round_store(mine, (const T*)nullptr);
      const float loss = logf(se) - (zy - zmax);
      if (lane == 0) a.row_loss[r] = loss;
      bad |= !isfinite(loss);
    }
  }
  if (bad && lane == 0) ri->diverged = 1;
  __syncthreads();
  // ---- delta of the layer below: a thread keeps the weights of 8 features in registers
  if (has_dgrad) {
    T* out = (T*)a.delta_in;
    int per = 1;
    while (per < nvec && per < 256) per <<= 1;
    const int nrl = 256 / per, rl = tid / per;
    for (int v0 = 0; v0 < nvec; v0 += per) {
      const int v = v0 + tid % per;
      if (v < nvec) {
        float wr[CC][8];
#pragma unroll
        for (int c = 0; c < CC; ++c) load8(wf + (size_t)c * wld + v * 8, wr[c]);
        for (int rr = rl; rr < R; rr += nrl) {
          float hv[8], acc8[8];
          load8(hs + (size_t)rr * in + v * 8, hv);
#pragma unroll
          for (int j = 0; j < 8; ++j) acc8[j] = 0.f;
#pragma unroll
          for (int c = 0; c < CC; ++c) {
            const float dv = d3[rr * CC + c];
#pragma unroll
            for (int j = 0; j < 8; ++j) acc8[j] = fmaf(dv, wr[c][j], acc8[j]);
          }
#pragma unroll
          for (int j = 0; j < 8; ++j) acc8[j] = hv[j] > 0.f ? acc8[j] : 0.f;
          store8(out + (size_t)(r0 + rr) * in + (size_t)v * 8, acc8);
        }
      }
    }
  }
  // ---- this block's share of the weight and bias gradient, staged in the (no longer needed)
  // transposed-weight area in the layout of the result and then copied out with coalesced stores
  float* dst = part + (size_t)blockIdx.x * (size_t)(in + 1) * CC;
  __syncthreads();                              // all reads of the transposed weights are done
  float* stg = wf;                              // [(in + 1)][CC]
  for (int it = tid; it < in / 2; it += 256) {
    const int m = 2 * it;
    float acc0[CC], acc1[CC];
#pragma unroll
    for (int c = 0; c < CC; ++c) { acc0[c] = 0.f; acc1[c] = 0.f; }
#pragma unroll 4
    for (int rr = 0; rr < R; ++rr) {
      float x0, x1;
      load2(hs + (size_t)rr * in + m, x0, x1);
#pragma unroll
      for (int c = 0; c < CC; ++c) {
        const float dv = d3[rr * CC + c];
        acc0[c] = fmaf(x0, dv, acc0[c]);
        acc1[c] = fmaf(x1, dv, acc1[c]);
      }
    }
#pragma unroll
    for (int c = 0; c < CC; ++c) { stg[m * CC + c] = acc0[c]; stg[(m + 1) * CC + c] = acc1[c]; }
  }
  if (tid < CC) {
    float tot = 0.f;
    for (int rr = 0; rr < R; ++rr) tot += d3[rr * CC + tid];
    stg[in * CC + tid] = tot;
  }
  __syncthreads();
  for (int i = tid; i < (in + 1) * CC; i += 256) dst[i] = stg[i];
}

// ---------------------------------------------------------------------------------------------
// Least squares, HBM-bound form (feature count a multiple of 8, at most LSQ_MAX_D).  Persistent
// CTAs take selected workers i = cta, cta + grid, ...; for each they draw the minibatch, compute
// the residuals r_b = x_b . w_v - y_b with 16-byte loads (one warp per row) and then add
// sum_b r_b x_b into register accumulators that persist across the CTA's workers (the second pass
// over the rows hits L2).  Eq. 3 only needs the sum over workers, so a CTA writes one partial sum.
constexpr int LSQ_MAX_D = 8192;

// NV = 16-byte vectors of the gradient a thread owns (d <= NV * 2048); wf[d] is dynamic shared memory.
template <typename T, int NV>
__global__ void __launch_bounds__(256, 2) lsq_grad_v2_kernel(LsqArgs a) {
  grid_dependency_sync();
  extern __shared__ __align__(16) float wf[];
  __shared__ float res[1024];
  __shared__ int sidx[1024];
  __shared__ float red[8];
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int K = ri->K, B = st->B, d = a.d, W = st->W, S = st->S, t = ri->t;
  const i64 M = st->n_samples;
  const uint32_t key0 = st->key0, key1 = st->key1;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = d >> 3;
  const T* X = (const T*)a.X;
  float acc[NV][8];
#pragma unroll
  for (int q = 0; q < NV; ++q)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[q][j] = 0.f;
  int slot_loaded = -1;
  bool bad = false;
  for (int i = blockIdx.x; i < K; i += gridDim.x) {
    const int wn = a.sel[i];
    const int job = a.job[wn];
    const int slot = (t - a.sel_tau[i]) % (S + 1);
    __syncthreads();                           // previous worker's res / sidx / wf are no longer read
    {
      const i64 lo = ((i64)wn * M) / W, hi = ((i64)(wn + 1) * M) / W;
      const u64 len = (u64)(hi - lo);
      for (int blk = tid; blk < ((B + 3) >> 2); blk += 256) {
        uint32_t w4[4];
        philox4x32_10((uint32_t)wn, (uint32_t)job, 1u, (uint32_t)blk, key0, key1, w4);
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (blk * 4 + q < B) sidx[blk * 4 + q] = (int)lo + (int)(((u64)w4[q] * len) >> 32);
      }
    }
    if (slot != slot_loaded) {
      const T* w = (const T*)a.ring + (size_t)slot * a.slot_stride;
      for (int v = tid; v < nvec; v += 256) {
        float wv[8];
        load8(w + v * 8, wv);
#pragma unroll
        for (int j = 0; j < 8; ++j) wf[v * 8 + j] = wv[j];
      }
      slot_loaded = slot;
    }
    __syncthreads();
    // pass 1: residuals; a warp takes two rows at a time and keeps 16 loads in flight per lane
    for (int b = warp; b < B; b += 16) {
      const int b2 = b + 8;
      const bool two = b2 < B;
      const T* x0 = X + (size_t)sidx[b] * d;
      const T* x1 = X + (size_t)sidx[two ? b2 : b] * d;
      float dot0 = 0.f, dot1 = 0.f;
#pragma unroll 8
      for (int v = lane; v < nvec; v += 32) {
        float xa[8], xb[8];
        load8(x0 + v * 8, xa);
        load8(x1 + v * 8, xb);
        const float4 w0 = *reinterpret_cast<const float4*>(wf + v * 8), w1 = *reinterpret_cast<const float4*>(wf + v * 8 + 4);
        dot0 = fmaf(xa[0], w0.x, dot0); dot0 = fmaf(xa[1], w0.y, dot0); dot0 = fmaf(xa[2], w0.z, dot0); dot0 = fmaf(xa[3], w0.w, dot0);
        dot0 = fmaf(xa[4], w1.x, dot0); dot0 = fmaf(xa[5], w1.y, dot0); dot0 = fmaf(xa[6], w1.z, dot0); dot0 = fmaf(xa[7], w1.w, dot0);
        dot1 = fmaf(xb[0], w0.x, dot1); dot1 = fmaf(xb[1], w0.y, dot1); dot1 = fmaf(xb[2], w0.z, dot1); dot1 = fmaf(xb[3], w0.w, dot1);
        dot1 = fmaf(xb[4], w1.x, dot1); dot1 = fmaf(xb[5], w1.y, dot1); dot1 = fmaf(xb[6], w1.z, dot1); dot1 = fmaf(xb[7], w1.w, dot1);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        dot0 += __shfl_xor_sync(0xffffffffu, dot0, o);
        dot1 += __shfl_xor_sync(0xffffffffu, dot1, o);
      }
      if (lane == 0) {
        res[b] = dot0 - a.y[sidx[b]];
        if (two) res[b2] = dot1 - a.y[sidx[b2]];
      }
    }
    __syncthreads();
    float part = 0.f;
    for (int b = tid; b < B; b += 256) part += 0.5f * res[b] * res[b];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if (lane == 0) red[warp] = part;
    // pass 2: this worker's gradient into the running sums (rows come from L2 now), with the
    // weight of its staleness when the staleness-aware step size is on
    const float sa = st->sa_penalty ? sa_weight(a.sel_tau[i]) : 1.f;
#pragma unroll
    for (int q = 0; q < NV; ++q) {
      const int v = tid + q * 256;
      if (v < nvec) {
#pragma unroll 8
        for (int b = 0; b < B; ++b) {
          float xv[8];
          load8(X + (size_t)sidx[b] * d + (size_t)v * 8, xv);
          const float rb = res[b] * sa;
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[q][j] = fmaf(rb, xv[j], acc[q][j]);
        }
      }
    }
    __syncthreads();
    if (tid == 0) {
      float tot = 0.f;
      for (int q = 0; q < 8; ++q) tot += red[q];
      const float loss = __fdiv_rn(tot, (float)B);
      a.loss[i] = loss;
      bad |= !isfinite(loss);
    }
  }
  if (bad) ri->diverged = 1;
  float* g = a.G + (size_t)blockIdx.x * a.slot_stride;
#pragma unroll
  for (int q = 0; q < NV; ++q) {
    const int v = tid + q * 256;
    if (v < nvec) store8(g + (size_t)v * 8, acc[q]);
  }
}

struct LsqUpdateArgs {
  const DevState* st;
  RoundInfo* ri;
  const int* job; u64* next_dur; int* dur_job;
  float* master; void* ring; const float* G;
  size_t d_pad; int d; int P; float lr;
  // when the gradient kernel leaves per-item loss sums (worker i, row group g): this kernel
  // finishes the uploaded losses loss[i] = (sum_g loss_part[i * groups + g]) / B
  const float* loss_part; float* loss; int groups;
};

// Eq. 3 for least squares: the P per-CTA partial sums are added in a fixed order (32 parameters x
// 8 partial lanes per block), then w^{t+1} = w^t - eta/(K B) * sum goes to the fp32 master and to
// ring slot (t+1) mod (S+1).
template <typename T>
__global__ void __launch_bounds__(256) lsq_update_kernel(LsqUpdateArgs a) {
  grid_dependency_sync();
  __shared__ float red[8][33];
  const DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  // duration look-ahead for the workers whose job index moved (first warp of the first ceil(N/32) blocks)
  if (a.next_dur != nullptr && threadIdx.x < 32 && (int)blockIdx.x * 32 < st->W)
    refresh_next_durations(st, a.job, a.next_dur, a.dur_job, (int)blockIdx.x * 32 + (int)threadIdx.x);
  if (ri->diverged) return;
  const int K = ri->K;
  if (a.loss_part != nullptr) {
    // every block adds the loss sums up the same way, so all of them agree on whether a
    // non-finite loss was uploaded (then Eq. 3 is not applied); block 0 publishes the losses
    bool bad = false;
    for (int i = threadIdx.x; i < K; i += 256) {
      float s = 0.f;
      for (int g = 0; g < a.groups; ++g) s += a.loss_part[(size_t)i * a.groups + g];
      const float loss = __fdiv_rn(s, (float)st->B);
      if (blockIdx.x == 0) a.loss[i] = loss;
      bad |= !isfinite(loss);
    }
    if (__syncthreads_or(bad ? 1 : 0)) {
      if (blockIdx.x == 0 && threadIdx.x == 0) ri->diverged = 1;
      return;
    }
  }
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int j = blockIdx.x * 32 + lane;
  float acc = 0.f;
  if (j < a.d) {
#pragma unroll 8
    for (int p = w; p < a.P; p += 8) acc += a.G[(size_t)p * a.d_pad + j];
  }
  red[w][lane] = acc;
  __syncthreads();
  if (w == 0 && j < a.d) {
    float g = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) g += red[q][lane];
    const float step = __fdiv_rn(a.lr, (float)(K * st->B));
    const float m = fmaf(-step, g, a.master[j]);
    a.master[j] = m;
    const int slot = (ri->t + 1) % (st->S + 1);
    stf((T*)a.ring + (size_t)slot * a.d_pad, j, m);
  }
}

}  // namespace absb
